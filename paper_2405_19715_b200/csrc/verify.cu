// Direct verify/correct kernel: one CTA per (row, position) unit, logits read with plain
// (vectorised where aligned) global loads.  Serves every shape, including rows that are not
// 16-byte aligned; the streaming kernel in verify_stream.cu is the fast path for large,
// aligned problems.  Operation: Algorithm 2 of arXiv 2405.19715 (see specdec.h).
#include "verify_unit.cuh"

namespace {

using namespace sd;


// DIRECT_THREADS threads per unit: 512 (two CTAs per SM) while the grid fills the machine less than
// twice, 256 (four per SM) beyond that, where more resident units hide each unit's dependent chain
// (accept test, draw, row counter) and pack the last wave better than a shorter pass does.
template <typename T, bool VEC, int DIRECT_THREADS>
__global__ void __launch_bounds__(DIRECT_THREADS, 1024 / DIRECT_THREADS) verify_direct_kernel(const VerifyParams P) {
    extern __shared__ float slab_sum[];
    __shared__ UnitShared sh;
    direct_unit<T, VEC, DIRECT_THREADS>(P, slab_sum, sh);
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
    const bool small_ctas = grid >= 4 * sms;
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
