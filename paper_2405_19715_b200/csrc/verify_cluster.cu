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
#include "verify_cluster.cuh"

namespace {

using namespace sd;

constexpr int CL_THREADS = 512;

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
    // length and drafted token are requested together; once they are known CTA 0 starts asynchronous
    // copies of the accept test's uniform and of the drafted token's two logits into shared memory,
    // every CTA one of the uniform of the draw
    u.L = P.lens ? ld_early_s32(P.lens + u.b) : P.K;
    int y = 0;
    if (rank == 0 && tid == 0 && u.i < P.K) y = ld_early_s32(P.tokens + (size_t)u.b * P.K + u.i);
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
    if (tid == 0) {
        const float* ur = P.uniforms + (size_t)u.b * (P.K + 1);
        scalar_fetch(&sh.pre[3], ur + P.K);
        if (rank == 0 && !u.bonus) {
            scalar_fetch(&sh.pre[0], ur + u.i);
            y_ok = (y >= 0 && y < P.V);
            if (y_ok) { logit_fetch(&sh.pre[1], trow, y); logit_fetch(&sh.pre[2], drow, y); }
        }
    }

    // ---- statistics of the slice
    Acc ap = acc_init(), aq = acc_init();
    unit_stats<T, VEC, CL_THREADS>(ts, ds, len, P.c, u.bonus, tid, ap, aq);
    if (tid == 0) scalars_wait();
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
            const float r = __uint_as_float(sh.pre[0]);
            const float t_y = logit_fetched(sh.pre[1], trow, y), d_y = logit_fetched(sh.pre[2], drow, y);
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
    int tok = -1;
    double W = 0.0;
    const float u01 = __uint_as_float(sh.pre[3]);
    if (cluster_draw<T, VEC, CL_THREADS>(Ps, ts, ds, start, len, mode, u01, sh.np, sh.nq, C, rank, cs, slab_sum, &tok, &W))
        unit_finish(P, u, 1, tok, (float)W, lane);
}

template <typename T>
cudaError_t launch_t(const VerifyParams& p, int C, cudaStream_t s) {
    constexpr int N = Elem<T>::EPV;
    const bool vec = (p.V % N == 0) && (reinterpret_cast<uintptr_t>(p.target) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(p.draft) % 16 == 0);
    const int slice_len = cluster_slice_len<T>(p.V, C);
    const size_t smem = (size_t)(slice_len / (32 * N)) * sizeof(float);
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
