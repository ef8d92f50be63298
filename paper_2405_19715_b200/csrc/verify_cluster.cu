// Verify/correct (Algorithm 2 of arXiv 2405.19715) for small batches: with only a few (row,
// position) units -- one sequence being decoded, a handful of candidates -- one CTA per unit
// leaves most SMs idle and each CTA walks its two logit rows in many dependent round trips.  Here a
// thread-block cluster of C CTAs shares a unit: CTA r takes the r-th contiguous slice of the
// vocabulary, so a row is covered in 1/C of the round trips, and the pieces are combined through
// distributed shared memory:
//
//   statistics of the slices  -> merged in rank order by every CTA (identical results);
//   accept test by CTA 0      -> its decision read by the others;
//   slice masses of the weights y' is drawn from -> every CTA finds the slice that holds u * W;
//   that CTA walks its slice and finishes the unit (row counter, first rejection, outputs).
//
// Every CTA of a cluster executes the same sequence of cluster barriers; early exits depend on the
// unit only, so they are taken by the whole cluster.
#include "verify_device.cuh"

namespace {

using namespace sd;

constexpr int CL_THREADS = 512;
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

template <typename T, bool VEC>
__global__ void __launch_bounds__(CL_THREADS) verify_cluster_kernel(const VerifyParams P, int C, int slice_len) {
    constexpr int N = Elem<T>::EPV;
    extern __shared__ float slab_sum[];
    __shared__ UnitShared sh;
    __shared__ ClusterShared cs;

    const uint32_t rank = cl_rank();
    const int unit = blockIdx.x / C;               // position-major, as in the one-CTA-per-unit kernel
    Unit u;
    u.i = unit / P.B;
    u.b = unit - u.i * P.B;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // length, uniform and drafted token are requested together; the drafted token's two logits
    // right behind the first row loads
    u.L = P.lens ? ld_early_s32(P.lens + u.b) : P.K;
    float r = 0.f;
    int y = 0;
    if (rank == 0 && tid == 0 && u.i < P.K) {
        r = ld_early_f32(P.uniforms + (size_t)u.b * (P.K + 1) + u.i);
        y = ld_early_s32(P.tokens + (size_t)u.b * P.K + u.i);
    }
    if (u.L < 0 || u.L > P.K) {                    // bad length: the row reports -1, nothing is read
        if (u.i == 0 && rank == 0 && tid == 0) {
            atomicOr(P.status, SPECDEC_DATA_BAD_LENGTH);
            P.n_acc[u.b] = -1;
            P.next[u.b] = -1;
            if (P.rmass) P.rmass[u.b] = 0.f;
        }
        return;
    }
    if (u.i > u.L) return;
    u.bonus = (u.i == u.L);

    const size_t V = (size_t)P.V;
    const T* trow = static_cast<const T*>(P.target) + ((size_t)u.b * (P.K + 1) + u.i) * V;
    const T* drow = u.bonus ? trow : static_cast<const T*>(P.draft) + ((size_t)u.b * P.K + u.i) * V;
    // this CTA's slice of the vocabulary
    const int start = min((int)rank * slice_len, P.V);
    const int len = min(slice_len, P.V - start);
    const T* ts = trow + start;
    const T* ds = drow + start;
    VerifyParams Ps = P;                           // the slice as a row of its own for the helpers
    Ps.V = len;

    int y_ok = 1;
    float t_y = 0.f, d_y = 0.f;
    auto gather_y = [&]() {
        if (rank == 0 && tid == 0 && !u.bonus) {
            y_ok = (y >= 0 && y < P.V);
            if (y_ok) { t_y = ld_early_logit(trow + y); d_y = ld_early_logit(drow + y); }
        }
    };

    // ---- statistics of the slice
    Acc ap = acc_init(), aq = acc_init();
    unit_stats<T, VEC, CL_THREADS>(ts, ds, len, P.c, u.bonus, tid, ap, aq, gather_y);
    warp_merge2(ap, aq);
    if (lane == 0) { sh.wp[warp] = ap; sh.wq[warp] = aq; }
    __syncthreads();
    if (warp == 0) {
        constexpr int NW = CL_THREADS / 32;
        Acc a = lane < NW ? sh.wp[lane] : acc_init(), b = lane < NW ? sh.wq[lane] : acc_init();
        warp_merge2(a, b);
        if (lane == 0) { cs.part_p = a; cs.part_q = b; }
    }
    cl_sync();                                     // every slice's statistics are in place

    // ---- merged statistics (rank order, the same in every CTA), accept test by CTA 0
    if (warp == 0) {
        Acc mp = acc_init(), mq = acc_init();
        if (lane < C) {
            mp.rs = cl_ld_f32(cl_map(&cs.part_p.rs, lane));
            mp.s = cl_ld_f32(cl_map(&cs.part_p.s, lane));
            mq.rs = cl_ld_f32(cl_map(&cs.part_q.rs, lane));
            mq.s = cl_ld_f32(cl_map(&cs.part_q.s, lane));
        }
        Acc gp = acc_init(), gq = acc_init();
        for (int k = 0; k < C; ++k) {
            Acc b;
            b.rs = __shfl_sync(0xffffffffu, mp.rs, k);
            b.s = __shfl_sync(0xffffffffu, mp.s, k);
            gp = acc_merge(gp, b);
            b.rs = __shfl_sync(0xffffffffu, mq.rs, k);
            b.s = __shfl_sync(0xffffffffu, mq.s, k);
            gq = acc_merge(gq, b);
        }
        if (rank == 0) {
            const int mode = unit_decide(P, u, gp, gq, t_y, d_y, y_ok, r, lane);
            if (lane == 0) cs.mode = mode;
        }
        if (lane == 0) {
            sh.np = make_norm(gp);
            sh.nq = u.bonus ? sh.np : make_norm(gq);
        }
    }
    cl_sync();                                     // CTA 0's decision is in place
    if (tid == 0) cs.mode_l = cl_ld_s32(cl_map(&cs.mode, 0));
    __syncthreads();
    int mode = cs.mode_l;
    if (mode == 0) {                               // cluster-uniform
        if (rank == 0 && warp == 0) unit_finish(P, u, 0, -1, 0.f, lane);
        cl_sync();                                 // CTA 0 stays until its decision has been read
        return;
    }

    // ---- the draw: slice masses, the slice that holds u * W, a walk inside it
    const int nvec = (len + N - 1) / N, nslab = (nvec + 31) / 32;
    double W_report = 0.0;
    for (int pass = 0; pass < 2; ++pass) {
        unit_slabs<T, VEC>(Ps, ts, ds, mode, sh.np, sh.nq, slab_sum, tid, CL_THREADS);
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
    if (warp == 0) {
        const double m = lane < C ? cl_ld_f64(cl_map(&cs.total, lane)) : 0.0;
        const float u01 = P.uniforms[(size_t)u.b * (P.K + 1) + P.K];
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
            const int tok = draw_select<T, VEC>(Ps, ts, ds, mode, u01, sh.np, sh.nq, slab_sum, lane, &total,
                                                tau > 0.0 ? tau : 0.0);
            unit_finish(P, u, 1, start + tok, (float)W_report, lane);
        }
    }
    cl_sync();                                     // nobody leaves while its mass may still be read
}

template <typename T>
cudaError_t launch_t(const VerifyParams& p, int C, cudaStream_t s) {
    constexpr int N = Elem<T>::EPV;
    const bool vec = (p.V % N == 0) && (reinterpret_cast<uintptr_t>(p.target) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(p.draft) % 16 == 0);
    // slices of whole slabs (32 vectors), so that a slice is as well aligned as the row
    const int nvec = (p.V + N - 1) / N;
    const int slabs = (nvec + 31) / 32, slab_per = (slabs + C - 1) / C;
    const int slice_len = slab_per * 32 * N;
    const size_t smem = (size_t)slab_per * sizeof(float);
    auto kern = vec ? verify_cluster_kernel<T, true> : verify_cluster_kernel<T, false>;
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * (p.K + 1) * C));
    cfg.blockDim = dim3(CL_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p, C, slice_len);
}

}  // namespace

int verify_cluster_size(const VerifyParams& p, specdec_dtype dtype, int sm_count) {
    const int units = p.B * (p.K + 1);
    const int nvec = p.V / (dtype == SPECDEC_BF16 ? 8 : 4);
    for (int C = CL_MAX; C >= 2; C >>= 1)
        if (units * C <= 2 * sm_count && nvec / C >= 2 * CL_THREADS) return C;   // a slice still gives every thread two vectors
    return 1;
}

cudaError_t launch_verify_cluster(const VerifyParams& p, specdec_dtype dtype, int C, cudaStream_t s, int* n_launch) {
    *n_launch = 1;
    return dtype == SPECDEC_BF16 ? launch_t<__nv_bfloat16>(p, C, s) : launch_t<float>(p, C, s);
}
