// Direct verify/correct kernel: one CTA per (row, position) unit, logits read with plain
// (vectorised where aligned) global loads.  Serves every shape, including rows that are not
// 16-byte aligned; the streaming kernel in verify_stream.cu is the fast path for large,
// aligned problems.  Operation: Algorithm 2 of arXiv 2405.19715 (see specdec.h).
#include "verify_device.cuh"

namespace {

using namespace sd;


// DIRECT_THREADS threads per unit: 512 (two CTAs per SM) when the units fit the machine a few times
// over, 256 (four per SM) for larger grids, where more resident units hide each unit's dependent
// chain (accept test, draw, row counter) better than a shorter pass does.
template <typename T, bool VEC, int DIRECT_THREADS>
__global__ void __launch_bounds__(DIRECT_THREADS, 1024 / DIRECT_THREADS) verify_direct_kernel(const VerifyParams P) {
    constexpr int N = Elem<T>::EPV;
    extern __shared__ float slab_sum[];
    __shared__ UnitShared sh;

    // position-major unit order: earlier positions of every row are scheduled first, so their
    // accept flags are usually known by the time a later position decides whether to draw
    const int unit = blockIdx.x;
    Unit u;
    u.i = unit / P.B;
    u.b = unit - u.i * P.B;
    u.L = P.lens ? P.lens[u.b] : P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (u.L < 0 || u.L > P.K) {                  // bad length: the row reports -1, nothing is read
        if (u.i == 0 && tid == 0) {
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

    // everything the accept test needs besides the sums is requested now and arrives during pass 1
    int y_ok = 1;
    float t_y = 0.f, d_y = 0.f, r = 0.f;
    if (tid == 0 && !u.bonus) {
        r = P.uniforms[(size_t)u.b * (P.K + 1) + u.i];
        const int y = P.tokens[(size_t)u.b * P.K + u.i];
        y_ok = (y >= 0 && y < P.V);
        if (y_ok) { t_y = to_float(trow[y]); d_y = to_float(drow[y]); }
    }

    // ---- pass 1: softmax statistics of both rows
    const int nvec = (P.V + N - 1) / N;
    Acc ap = acc_init(), aq = acc_init();
    unit_stats<T, VEC, DIRECT_THREADS>(trow, drow, P.V, P.c, u.bonus, tid, ap, aq);
    ap = warp_merge(ap);
    aq = warp_merge(aq);
    if (lane == 0) { sh.wp[warp] = ap; sh.wq[warp] = aq; }
    __syncthreads();
    if (warp == 0) {
        constexpr int NW = DIRECT_THREADS / 32;
        Acc a = lane < NW ? sh.wp[lane] : acc_init(), b = lane < NW ? sh.wq[lane] : acc_init();
        a = warp_merge(a);
        b = warp_merge(b);
        const int mode = unit_decide(P, u, a, b, t_y, d_y, y_ok, r, lane);
        if (lane == 0) {
            sh.np = make_norm(a);
            sh.nq = u.bonus ? sh.np : make_norm(b);
            sh.need_draw = mode;
        }
    }
    __syncthreads();

    // ---- pass 2 (only where this position may supply y'): weights, prefix, inverse CDF
    const int mode = sh.need_draw;
    if (mode) {
        const float u01 = P.uniforms[(size_t)u.b * (P.K + 1) + P.K];
        unit_draw<T, VEC>(P, trow, drow, mode, u01, sh, slab_sum, tid, DIRECT_THREADS, 0);
        if (mode == 1 && !(sh.total > 1e-30)) {   // p == q to rounding: draw from p itself
            const double keep = sh.total;
            __syncthreads();
            unit_draw<T, VEC>(P, trow, drow, 2, u01, sh, slab_sum, tid, DIRECT_THREADS, 0);
            if (tid == 0) sh.total = keep;
            __syncthreads();
        }
    }
    if (warp == 0) unit_finish(P, u, mode != 0, sh.token, mode ? (float)sh.total : 0.f, lane);
}

template <typename T>
cudaError_t launch_t(const VerifyParams& p, cudaStream_t s) {
    constexpr int N = Elem<T>::EPV;
    const int nvec = (p.V + N - 1) / N;
    const int nslab = (nvec + 31) / 32;
    const size_t smem = (size_t)nslab * sizeof(float);
    const bool vec = (p.V % N == 0) && (reinterpret_cast<uintptr_t>(p.target) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(p.draft) % 16 == 0);
    const int grid = p.B * (p.K + 1);
    static const int sms = [] {
        int dev = 0, n = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        return n;
    }();
    const bool small_ctas = grid >= 12 * sms;
    auto kern = small_ctas ? (vec ? verify_direct_kernel<T, true, 256> : verify_direct_kernel<T, false, 256>)
                           : (vec ? verify_direct_kernel<T, true, 512> : verify_direct_kernel<T, false, 512>);
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<grid, small_ctas ? 256 : 512, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_verify_direct(const VerifyParams& p, specdec_dtype dtype, cudaStream_t s, int* n_launch) {
    *n_launch = 1;
    return dtype == SPECDEC_BF16 ? launch_t<__nv_bfloat16>(p, s) : launch_t<float>(p, s);
}
