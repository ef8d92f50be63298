// Greedy verification (Section 4.1 of arXiv 2405.19715): with greedy decoding a drafted token is
// kept while it equals the target model's argmax at its position; the first mismatch is replaced
// by that argmax, and when all candidates match the target's argmax at the next position is
// appended.  Only target rows are read: one CTA per (row, position <= L) finds the row's argmax
// (lowest index on ties), the last position of a row to finish ballots the matches.
#include "verify_device.cuh"

namespace {

using namespace sd;

constexpr int GREEDY_THREADS = 256;

struct Best {
    float v;
    int i;
};
__device__ __forceinline__ Best better(const Best& a, const Best& b) {      // larger value, then lower index
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(GREEDY_THREADS) greedy_kernel(const VerifyParams P, int32_t* __restrict__ argmax_out) {
    constexpr int N = Elem<T>::EPV;
    __shared__ Best wbest[GREEDY_THREADS / 32];
    const int unit = blockIdx.x;
    Unit u;
    u.i = unit / P.B;
    u.b = unit - u.i * P.B;
    u.L = P.lens ? P.lens[u.b] : P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (u.L < 0 || u.L > P.K) {
        if (u.i == 0 && tid == 0) {
            atomicOr(P.status, SPECDEC_DATA_BAD_LENGTH);
            P.n_acc[u.b] = -1;
            P.next[u.b] = -1;
        }
        if (argmax_out && tid == 0) argmax_out[(size_t)u.b * (P.K + 1) + u.i] = -1;
        return;
    }
    if (u.i > u.L) {
        if (argmax_out && tid == 0) argmax_out[(size_t)u.b * (P.K + 1) + u.i] = -1;
        return;
    }
    u.bonus = (u.i == u.L);
    const T* row = static_cast<const T*>(P.target) + ((size_t)u.b * (P.K + 1) + u.i) * (size_t)P.V;
    const int nvec = (P.V + N - 1) / N;
    Best best{-INFINITY, 0x7fffffff};
    if constexpr (VEC) {
        constexpr int U = 4;
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        const uint32_t ninf = neg_inf_word(T());
        for (int j0 = tid; j0 < nvec; j0 += U * GREEDY_THREADS) {
            uint4 r[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = j0 + k * GREEDY_THREADS;
                r[k] = j < nvec ? __ldcg(rv + j) : make_uint4(ninf, ninf, ninf, ninf);
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const float m = vec_max(r[k], T());
                if (m > best.v) {                       // strict: an equal value later in the row never wins
                    float x[N];
                    unpack(r[k], x);
                    int at = 0;
#pragma unroll
                    for (int e = N - 1; e >= 0; --e)
                        if (x[e] == m) at = e;
                    best = Best{m, (j0 + k * GREEDY_THREADS) * N + at};
                }
            }
        }
    } else {
        for (int v = tid; v < P.V; v += GREEDY_THREADS) {
            const float x = to_float(row[v]);
            if (x > best.v) best = Best{x, v};
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Best other{__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
        best = better(best, other);
    }
    if (lane == 0) wbest[warp] = best;
    __syncthreads();
    if (warp != 0) return;
    best = lane < GREEDY_THREADS / 32 ? wbest[lane] : Best{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Best other{__shfl_xor_sync(0xffffffffu, best.v, o), __shfl_xor_sync(0xffffffffu, best.i, o)};
        best = better(best, other);
    }
    const int am = best.i == 0x7fffffff ? 0 : best.i;       // a row of NaN / -inf only: token 0
    if (lane == 0) {
        if (argmax_out) argmax_out[(size_t)u.b * (P.K + 1) + u.i] = am;
        st_relaxed(&P.draws[(size_t)u.b * (P.K + 1) + u.i], am);
        if (!u.bonus) {
            const int y = P.tokens[(size_t)u.b * P.K + u.i];
            const int state = (y < 0 || y >= P.V) ? FLAG_BAD : (y == am ? FLAG_ACCEPT : FLAG_REJECT);
            if (state == FLAG_BAD) atomicOr(P.status, SPECDEC_DATA_BAD_TOKEN);
            st_relaxed(&P.flags[(size_t)u.b * P.K + u.i], (int)((P.epoch << 2) | (uint32_t)state));
        }
    }
    if (!row_arrive(P, u, lane)) return;
    int n, bad;
    row_resolve(P, u, lane, n, bad);
    if (lane == 0) {
        P.n_acc[u.b] = bad ? -1 : n;
        P.next[u.b] = bad ? -1 : ld_acquire(&P.draws[(size_t)u.b * (P.K + 1) + n]);
    }
}

}  // namespace

cudaError_t launch_greedy(const VerifyParams& p, specdec_dtype dtype, int32_t* argmax_out, cudaStream_t s) {
    const int es = dtype == SPECDEC_BF16 ? 2 : 4;
    const bool vec = ((size_t)p.V * es) % 16 == 0 && reinterpret_cast<uintptr_t>(p.target) % 16 == 0;
    const int grid = p.B * (p.K + 1);
    if (dtype == SPECDEC_BF16) {
        if (vec) greedy_kernel<__nv_bfloat16, true><<<grid, GREEDY_THREADS, 0, s>>>(p, argmax_out);
        else greedy_kernel<__nv_bfloat16, false><<<grid, GREEDY_THREADS, 0, s>>>(p, argmax_out);
    } else {
        if (vec) greedy_kernel<float, true><<<grid, GREEDY_THREADS, 0, s>>>(p, argmax_out);
        else greedy_kernel<float, false><<<grid, GREEDY_THREADS, 0, s>>>(p, argmax_out);
    }
    return cudaGetLastError();
}
