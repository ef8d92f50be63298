// Threshold stop rule (Section 4.3 and the loop of Algorithm 1, arXiv 2405.19715):
// p_hat <- p_hat * accept_prob[i]; stop at the first i with 1 - p_hat > h.
#include "specdec_internal.h"

namespace {

__global__ void stop_kernel(const float* __restrict__ a, const int32_t* __restrict__ lens, float h, int B, int K,
                            int32_t* __restrict__ stop_pos, uint32_t* __restrict__ status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int L = lens ? lens[b] : K;
    if (L < 0 || L > K) {                        // bad length: the row reports -1, nothing is read
        atomicOr(status, SPECDEC_DATA_BAD_LENGTH);
        stop_pos[b] = -1;
        return;
    }
    const float* row = a + (size_t)b * K;
    float c = 1.f;
    int pos = L;
    for (int j = 0; j < L; ++j) {
        c *= row[j];
        if (1.f - c > h) { pos = j; break; }
    }
    stop_pos[b] = pos;
}

// One trip of Algorithm 1's loop for every row: p_hat <- p_hat * a; stop iff 1 - p_hat > h.
__global__ void stop_step_kernel(const float* __restrict__ a, float* __restrict__ p_hat, float h, int B,
                                 int32_t* __restrict__ stop) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const float p = p_hat[b] * a[b];
    p_hat[b] = p;
    stop[b] = (1.f - p > h) ? 1 : 0;
}

}  // namespace

cudaError_t launch_stop_step(const float* accept_prob_step, float* p_hat, float h, int B, int32_t* stop,
                             cudaStream_t s) {
    stop_step_kernel<<<(B + 127) / 128, 128, 0, s>>>(accept_prob_step, p_hat, h, B, stop);
    return cudaGetLastError();
}

cudaError_t launch_stop(const float* accept_prob, const int32_t* lens, float h, int B, int K, int32_t* stop_pos,
                        uint32_t* status, cudaStream_t s) {
    const int threads = 128;
    stop_kernel<<<(B + threads - 1) / threads, threads, 0, s>>>(accept_prob, lens, h, B, K, stop_pos, status);
    return cudaGetLastError();
}
