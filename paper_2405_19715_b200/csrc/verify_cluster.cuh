// Pieces shared by the kernels that spread one row pair over a thread-block cluster
// (verify_cluster.cu: a whole unit per cluster; verify_split.cu: one draw per cluster): access to the
// other CTAs' shared memory and the inverse-CDF draw of Appendix C of arXiv 2405.19715 over a row pair
// whose vocabulary is cut into one slice per CTA.
#pragma once

#include "verify_device.cuh"

namespace sd {

constexpr int CL_MAX = 8;                          // portable cluster size limit

struct ClusterShared {
    Acc part_p, part_q;                            // this CTA's slice statistics
    double total;                                  // this CTA's slice mass
    double W;                                      // mass of the whole row (local copy)
    int mode;                                      // CTA 0: 0 no draw, 1 residual, 2 target itself
    int mode_l;                                    // local copy of CTA 0's decision
};

__device__ __forceinline__ uint32_t cl_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cl_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of `p` (own shared memory) as seen in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t cl_map(const void* p, uint32_t rank) {
    uint32_t a = (uint32_t)__cvta_generic_to_shared(p), r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
__device__ __forceinline__ float cl_ld_f32(uint32_t a) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ double cl_ld_f64(uint32_t a) {
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ int cl_ld_s32(uint32_t a) {
    int v;
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}

// Slices of whole slabs (32 vectors), so that a slice is as well aligned as the row it is cut from.
template <typename T>
__host__ __device__ inline int cluster_slice_len(int V, int C) {
    constexpr int N = Elem<T>::EPV;
    const int nvec = (V + N - 1) / N;
    const int slabs = (nvec + 31) / 32, slab_per = (slabs + C - 1) / C;
    return slab_per * 32 * N;
}

// The draw of y' by a cluster of C CTAs, CTA `rank` holding the slice [start, start + len) of the rows
// (`ts`, `ds` point at the slice; Ps is the problem with V = len).  Slice masses of the weights
// ((p - q)_+ for mode 1, p for mode 2) are exchanged through distributed shared memory, every CTA finds
// the slice that holds u01 * W, and that CTA alone walks its slice.  Returns true in warp 0 of the
// owning CTA (all its lanes), with the token (a vocabulary index) and the mass W the caller reports;
// false everywhere else.  If the residual has no mass (p == q to rounding) the draw is made from p
// itself and *W_out keeps the residual's mass.  Every CTA of the cluster must call, with all its
// threads; three or five cluster barriers are executed, the last one after every remote read.
template <typename T, bool VEC, int THREADS>
__device__ __forceinline__ bool cluster_draw(const VerifyParams& Ps, const T* __restrict__ ts, const T* __restrict__ ds,
                                             int start, int len, int mode, float u01, const Norm np, const Norm nq,
                                             int C, uint32_t rank, ClusterShared& cs, float* __restrict__ slab_sum,
                                             int* token_out, double* W_out) {
    constexpr int N = Elem<T>::EPV;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = (len + N - 1) / N, nslab = (nvec + 31) / 32;
    double W_report = 0.0;
    for (int pass = 0; pass < 2; ++pass) {
        unit_slabs<T, VEC>(Ps, ts, ds, mode, np, nq, slab_sum, tid, THREADS);
        __syncthreads();
        if (warp == 0) {
            const double tot = slab_total(slab_sum, nslab, lane);
            if (lane == 0) cs.total = tot;
        }
        cl_sync();                                 // every slice's mass is in place
        if (warp == 0) {
            const double m = lane < C ? cl_ld_f64(cl_map(&cs.total, lane)) : 0.0;
            double W = 0.0;
            for (int k = 0; k < C; ++k) W += __shfl_sync(0xffffffffu, m, k);
            if (lane == 0) cs.W = W;
        }
        __syncthreads();
        if (pass == 0) W_report = cs.W;
        if (pass == 0 && mode == 1 && !(cs.W > 1e-30)) {   // p == q to rounding: draw from p itself (cluster-uniform)
            mode = 2;
            cl_sync();                             // all masses have been read before they are overwritten
            continue;
        }
        break;
    }
    bool mine = false;
    if (warp == 0) {
        const double m = lane < C ? cl_ld_f64(cl_map(&cs.total, lane)) : 0.0;
        const double thr = (double)u01 * cs.W;
        int owner = -1, lastpos = -1;
        double before = 0.0, run = 0.0;
        for (int k = 0; k < C; ++k) {
            const double mk = __shfl_sync(0xffffffffu, m, k);
            if (mk > 0.0) lastpos = k;
            if (owner < 0 && run + mk > thr) { owner = k; before = run; }
            run += mk;
        }
        if (owner < 0) {                           // rounding left nothing above u * W: the last slice with mass
            owner = lastpos < 0 ? 0 : lastpos;
            before = 0.0;
            for (int k = 0; k < owner; ++k) before += __shfl_sync(0xffffffffu, m, k);
        }
        if (owner == (int)rank) {
            double total;
            const double tau = thr - before;
            const int tok = draw_select<T, VEC>(Ps, ts, ds, mode, u01, np, nq, slab_sum, lane, &total,
                                                tau > 0.0 ? tau : 0.0);
            *token_out = start + tok;
            *W_out = W_report;
            mine = true;
        }
    }
    cl_sync();                                     // nobody leaves while its mass may still be read
    return mine;
}

}  // namespace sd
