// Verify/correct under top-k sampling (Appendix D.1 of arXiv 2405.19715: the paper decodes with
// k = 50): both models' logits below the k-th largest of their row count as -inf, then Algorithm 2
// runs on the filtered distributions.
//
// Only about k logits per row matter, so nothing is exponentiated while streaming.  One CTA per
// (row, position), two passes per logit row:
//   1. every thread takes the maximum of its strided share of the row; the smallest, over warps, of
//      each warp's r-th largest thread maximum (r = ceil(k / warps)) is a lower bound on the k-th
//      largest of the row, and a tight one: a thread's share holds 1/512 of the row, so few of the
//      top k collide in one share;
//   2. the row is read again, newest lines first so that they still sit in L2, and every logit at or
//      above the bound goes into a candidate buffer in shared memory (k plus a few tens).
// The exact k-th largest is found among the candidates (rank counting, radix select when there are
// many), and the softmax terms, the accept test and -- for a rejecting or bonus position -- the
// residual draw are evaluated on the kept candidates in fp64 by the whole CTA.  If the bound turns
// out too loose for the buffer (rows with -inf or repeated maxima), an exact radix select over the
// row supplies the threshold and the row is filtered again.
#include "verify_device.cuh"

namespace {

using namespace sd;

constexpr int TK_THREADS = 512;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int CAP = 4096;                 // candidates per row; every V <= CAP fits whole
constexpr int MAX_KEPT = CAP / 2;         // kept entries (k + ties at the k-th value) the draw can hold
constexpr int RANK_COUNT_MAX = 1024;      // above this many candidates the k-th largest comes from a radix select

struct TkShared {
    float warp_rth[2][TK_WARPS];
    float bound[2], tau[2];
    int count[2], overflow[2];
    unsigned int hist[256];
    unsigned int sel_prefix, sel_rank;
    double zsum[2], dmax[2];
    int state, n_kept, token, retry;
    float mass;
};

__device__ __forceinline__ uint32_t order_key(float x) {        // larger float <-> larger key; NaN sorts lowest
    if (x != x) return 0u;
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// r-th largest of the 32 lane values (all lanes get it); -inf when fewer than r are above -inf.
__device__ __forceinline__ float warp_rth_largest(float v, int r, int lane) {
    float cur = -INFINITY;
    for (int it = 0; it < r; ++it) {
        float m;
        asm("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
        cur = m;
        const unsigned who = __ballot_sync(0xffffffffu, v == m);
        if (who == 0u) return -INFINITY;                        // only NaN left
        if (lane == __ffs(who) - 1) v = -INFINITY;
        if (m == -INFINITY) break;
    }
    return cur;
}

// Pass 1: this thread's maximum over its strided share of the row (NaN ignored).
template <typename T, bool VEC>
__device__ __forceinline__ float thread_max(const T* __restrict__ row, int V, int tid) {
    constexpr int N = Elem<T>::EPV;
    float m = -INFINITY;
    if constexpr (VEC) {
        constexpr int U = 4;
        const int nvec = V / N;
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        const uint32_t ninf = neg_inf_word(T());
        for (int j0 = tid; j0 < nvec; j0 += U * TK_THREADS) {
            uint4 r[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = j0 + k * TK_THREADS;
                r[k] = j < nvec ? __ldcg(rv + j) : make_uint4(ninf, ninf, ninf, ninf);
            }
#pragma unroll
            for (int k = 0; k < U; ++k) m = fmaxf(m, vec_max(r[k], T()));
        }
    } else {
        for (int v = tid; v < V; v += TK_THREADS) {
            const float x = to_float(row[v]);
            if (x == x) m = fmaxf(m, x);
        }
    }
    return m;
}

// Pass 2: every logit at or above the bound goes into the candidate buffer, last lines first.
template <typename T, bool VEC>
__device__ __forceinline__ void filter_row(const T* __restrict__ row, int V, float bound, float* cval, int* cidx,
                                           int* count, int* overflow, int tid) {
    constexpr int N = Elem<T>::EPV;
    if constexpr (VEC) {
        constexpr int U = 4;
        constexpr int STEP = U * TK_THREADS;
        const int nvec = V / N;
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        const uint32_t ninf = neg_inf_word(T());
        for (int base = ((nvec - 1) / STEP) * STEP; base >= 0; base -= STEP) {
            uint4 r[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = base + tid + k * TK_THREADS;
                r[k] = j < nvec ? __ldcg(rv + j) : make_uint4(ninf, ninf, ninf, ninf);
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = base + tid + k * TK_THREADS;
                if (j < nvec && vec_max(r[k], T()) >= bound) {
                    float x[N];
                    unpack(r[k], x);
#pragma unroll
                    for (int e = 0; e < N; ++e)
                        if (x[e] >= bound) {
                            const int pos = atomicAdd(count, 1);
                            if (pos < CAP) { cval[pos] = x[e]; cidx[pos] = j * N + e; }
                            else *overflow = 1;
                        }
                }
            }
        }
    } else {
        for (int v = tid; v < V; v += TK_THREADS) {
            const float x = to_float(row[v]);
            if (x >= bound) {
                const int pos = atomicAdd(count, 1);
                if (pos < CAP) { cval[pos] = x; cidx[pos] = v; }
                else *overflow = 1;
            }
        }
    }
}

// Exact k-th largest of n values by radix select on order-preserving keys, eight bits a pass.
// `at(i)` yields value i; every thread of the CTA calls it and gets the result.
template <typename F>
__device__ float radix_kth_largest(F at, int n, int k, TkShared& sh, int tid) {
    uint32_t prefix = 0, mask = 0;
    int rank = k;                                  // rank-th largest among keys matching the prefix
    const int lane = tid & 31;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += TK_THREADS) sh.hist[i] = 0;
        __syncthreads();
        for (int v = tid; v < n; v += TK_THREADS) {
            const uint32_t key = order_key(at(v));
            if ((key & mask) == prefix) atomicAdd(&sh.hist[(key >> shift) & 0xffu], 1u);
        }
        __syncthreads();
        if (tid < 32) {
            // lane l owns bins 255-8l down to 248-8l; counts above its bins by a warp scan
            int own = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) own += (int)sh.hist[255 - 8 * lane - q];
            int incl = own;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const int excl = incl - own;
            const bool mine = excl < rank && rank <= incl;
            const unsigned who = __ballot_sync(0xffffffffu, mine);
            if (who == 0u) {                       // fewer than rank keys left (cannot happen for k <= n)
                if (lane == 0) { sh.sel_prefix = prefix; sh.sel_rank = 1; }
            } else if (mine) {
                int r = rank - excl, bin = 255 - 8 * lane;
                for (int q = 0; q < 7; ++q, --bin) {           // the eighth bin takes what is left
                    const int h = (int)sh.hist[bin];
                    if (h >= r) break;
                    r -= h;
                }
                sh.sel_prefix = prefix | ((uint32_t)bin << shift);
                sh.sel_rank = (unsigned)r;
            }
        }
        __syncthreads();
        prefix = sh.sel_prefix;
        rank = (int)sh.sel_rank;
        mask |= 0xffu << shift;
        __syncthreads();
    }
    return key_to_float(prefix);
}

template <typename T, bool VEC>
__global__ void __launch_bounds__(TK_THREADS, 2) verify_topk_kernel(const VerifyParams P, int top_k) {
    extern __shared__ __align__(16) unsigned char tk_smem[];
    float* cval = reinterpret_cast<float*>(tk_smem);                   // [2][CAP]
    int* cidx = reinterpret_cast<int*>(tk_smem + 2 * CAP * sizeof(float));   // [2][CAP]
    __shared__ TkShared sh;

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
            if (P.rmass) P.rmass[u.b] = 0.f;
        }
        return;
    }
    if (u.i > u.L) return;
    u.bonus = (u.i == u.L);
    const int V = P.V;
    const T* rows[2];
    rows[0] = static_cast<const T*>(P.target) + ((size_t)u.b * (P.K + 1) + u.i) * (size_t)V;
    rows[1] = u.bonus ? rows[0] : static_cast<const T*>(P.draft) + ((size_t)u.b * P.K + u.i) * (size_t)V;
    const int nrows = u.bonus ? 1 : 2;
    const int k = min(top_k, V);

    // accept-test operands, requested early
    int y = 0, y_ok = 1;
    float t_y = 0.f, d_y = 0.f, r_acc = 0.f;
    if (tid == 0 && !u.bonus) {
        r_acc = P.uniforms[(size_t)u.b * (P.K + 1) + u.i];
        y = P.tokens[(size_t)u.b * P.K + u.i];
        y_ok = (y >= 0 && y < V);
        if (y_ok) { t_y = to_float(rows[0][y]); d_y = to_float(rows[1][y]); }
    }
    if (tid < 2) { sh.count[tid] = 0; sh.overflow[tid] = 0; }

    const int rth = (k + TK_WARPS - 1) / TK_WARPS;
    for (int rr = 0; rr < nrows; ++rr) {
        // ---- pass 1: a lower bound on the k-th largest of the row
        const float wr = warp_rth_largest(thread_max<T, VEC>(rows[rr], V, tid), rth, lane);
        if (lane == 0) sh.warp_rth[rr][warp] = wr;
        __syncthreads();
        float b = sh.warp_rth[rr][0];
#pragma unroll
        for (int w = 1; w < TK_WARPS; ++w) b = fminf(b, sh.warp_rth[rr][w]);
        // ---- pass 2: candidates at or above the bound
        float* cv = cval + rr * CAP;
        int* ci = cidx + rr * CAP;
        filter_row<T, VEC>(rows[rr], V, b, cv, ci, &sh.count[rr], &sh.overflow[rr], tid);
        __syncthreads();
        if (sh.overflow[rr]) {                         // block-uniform: the bound was too loose
            const T* row = rows[rr];
            const float kth = radix_kth_largest([row](int v) { return to_float(row[v]); }, V, k, sh, tid);
            if (tid == 0) { sh.count[rr] = 0; sh.overflow[rr] = 0; }
            __syncthreads();
            filter_row<T, VEC>(row, V, kth, cv, ci, &sh.count[rr], &sh.overflow[rr], tid);
            __syncthreads();
        }

        // ---- exact k-th largest among the candidates, softmax terms of the kept ones (fp64)
        const int n = min(sh.count[rr], CAP);
        const int kk = min(k, n);                      // n <= k: every candidate is kept, tau is their minimum
        float tau = -INFINITY;
        if (n > RANK_COUNT_MAX) {
            tau = radix_kth_largest([cv](int c) { return cv[c]; }, n, kk, sh, tid);
        } else if (n > 0) {
            if (tid == 0) sh.tau[rr] = -INFINITY;
            __syncthreads();
            for (int c = tid; c < n; c += TK_THREADS) {
                const float vc = cv[c];
                int gt = 0, ge = 0;
                for (int j = 0; j < n; ++j) { gt += cv[j] > vc; ge += cv[j] >= vc; }
                if (gt < kk && kk <= ge) sh.tau[rr] = vc;             // every such c carries the same value
            }
            __syncthreads();
            tau = sh.tau[rr];
        }
        float m = -INFINITY;
        for (int c = tid; c < n; c += TK_THREADS) if (cv[c] >= tau) m = fmaxf(m, cv[c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) sh.warp_rth[rr][warp] = m;
        if (tid == 0) { sh.tau[rr] = tau; sh.zsum[rr] = 0.0; }
        __syncthreads();
        float mm = sh.warp_rth[rr][0];
#pragma unroll
        for (int w = 1; w < TK_WARPS; ++w) mm = fmaxf(mm, sh.warp_rth[rr][w]);
        const double dm = (double)mm, cc = (double)P.c;
        double z = 0.0;
        for (int c = tid; c < n; c += TK_THREADS) if (cv[c] >= tau) z += exp2(((double)cv[c] - dm) * cc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        if (lane == 0 && z != 0.0) atomicAdd(&sh.zsum[rr], z);
        if (tid == 0) sh.dmax[rr] = dm;
        __syncthreads();
    }
    const bool too_many_ties = sh.overflow[0] || (nrows == 2 && sh.overflow[1]);

    // ---- accept test (thread 0)
    const double cc = (double)P.c;
    const float tau_p = sh.tau[0], tau_q = nrows == 2 ? sh.tau[1] : -INFINITY;
    const double mp = sh.dmax[0], zp = sh.zsum[0];
    const double mq = nrows == 2 ? sh.dmax[1] : 0.0, zq = nrows == 2 ? sh.zsum[1] : 1.0;
    if (tid == 0) {
        int state = 0;
        if (!u.bonus) {
            double ratio;
            const bool p_in = y_ok && t_y >= tau_p && t_y > -INFINITY, q_in = y_ok && d_y >= tau_q && d_y > -INFINITY;
            if (!p_in) ratio = 0.0;                                      // p'(y) = 0: certain rejection
            else if (!q_in) ratio = INFINITY;
            else ratio = exp2((((double)t_y - mp) - ((double)d_y - mq)) * cc) * (zq / zp);
            state = (!y_ok || too_many_ties) ? FLAG_BAD : ((double)r_acc >= ratio ? FLAG_REJECT : FLAG_ACCEPT);
            if (!y_ok) atomicOr(P.status, SPECDEC_DATA_BAD_TOKEN);
            if (P.ratio) P.ratio[(size_t)u.b * P.K + u.i] = state == FLAG_BAD ? -1.f : (float)fmin(1.0, ratio);
            st_relaxed(&P.flags[(size_t)u.b * P.K + u.i], (int)((P.epoch << 2) | (uint32_t)state));
        }
        if (too_many_ties) atomicOr(P.status, SPECDEC_DATA_TOPK_TIES);
        sh.state = state;
        sh.n_kept = 0;
        sh.token = -1;
        sh.mass = 0.f;
        sh.retry = 0;
    }
    __syncthreads();
    // a position whose draw cannot be made (ties beyond the buffers) records the token -1
    const bool draw = u.bonus || sh.state == FLAG_REJECT;

    // ---- the draw of a rejecting or bonus position: kept target candidates in vocabulary order with
    //      weights (p' - q')_+ (p' at the bonus position, or when p' = q' on the whole support)
    if (draw && !too_many_ties) {                      // block-uniform
        const int n = min(sh.count[0], CAP);
        int* ki = cidx + CAP;                          // the draft row's buffers are free to reuse now
        float* kv = cval + CAP;
        for (int c = tid; c < n; c += TK_THREADS)
            if (cval[c] >= tau_p) {
                const int pos = atomicAdd(&sh.n_kept, 1);
                if (pos < MAX_KEPT) { ki[pos] = cidx[c]; kv[pos] = cval[c]; }
            }
        __syncthreads();
        const int kept = sh.n_kept;
        if (kept > MAX_KEPT) {                         // thousands of ties at the k-th value
            if (tid == 0) atomicOr(P.status, SPECDEC_DATA_TOPK_TIES);
        } else {
            int* si = cidx;                            // sorted indices; the target's candidates are consumed
            double* sw = reinterpret_cast<double*>(cval);      // [MAX_KEPT] weights in vocabulary order
            const T* drow = rows[1];
            for (int pass = 0; pass < 2; ++pass) {
                const bool resid = !u.bonus && pass == 0;
                __syncthreads();
                for (int a = tid; a < kept; a += TK_THREADS) {
                    const int ia = ki[a];
                    int rank = 0;
                    for (int j = 0; j < kept; ++j) rank += ki[j] < ia;
                    double w = exp2(((double)kv[a] - mp) * cc) / zp;
                    if (resid) {
                        const float dv = to_float(drow[ia]);
                        const double qv = (dv >= tau_q && dv > -INFINITY) ? exp2(((double)dv - mq) * cc) / zq : 0.0;
                        w = fmax(w - qv, 0.0);
                    }
                    si[rank] = ia;
                    sw[rank] = w;
                }
                __syncthreads();
                if (warp == 0) {
                    // lane l sums entries [l*seg, (l+1)*seg); a warp scan gives the mass before each segment
                    const int seg = (kept + 31) / 32, a0 = min(lane * seg, kept), a1 = min(a0 + seg, kept);
                    double own = 0.0;
                    for (int a = a0; a < a1; ++a) own += sw[a];
                    double incl = own;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double t = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += t;
                    }
                    const double tot = __shfl_sync(0xffffffffu, incl, 31);
                    if (pass == 0 && lane == 0) sh.mass = u.bonus ? 1.f : (float)tot;
                    if (tot > 1e-30) {
                        const double thr = (double)P.uniforms[(size_t)u.b * (P.K + 1) + P.K] * tot;
                        const unsigned hit = __ballot_sync(0xffffffffu, incl > thr);
                        int lastpos = -1;
                        for (int a = a0; a < a1; ++a) if (sw[a] > 0.0) lastpos = a;
                        if (hit) {
                            if (lane == __ffs(hit) - 1) {
                                double run = incl - own;
                                int tok = -1;
                                for (int a = a0; a < a1; ++a) {
                                    run += sw[a];
                                    if (run > thr) { tok = si[a]; break; }
                                }
                                if (tok < 0 && lastpos >= 0) tok = si[lastpos];   // rounding at the segment's end
                                sh.token = tok;
                            }
                        } else {
                            // u * W rounds to W: the last entry with weight
                            const unsigned has = __ballot_sync(0xffffffffu, lastpos >= 0);
                            if (has && lane == 31 - __clz(has)) sh.token = si[lastpos];
                        }
                    } else if (lane == 0) {
                        sh.retry = (pass == 0 && !u.bonus);
                    }
                }
                __syncthreads();
                if (!sh.retry) break;                  // block-uniform; only ever set in pass 0
            }
        }
    }
    if (warp != 0) return;
    unit_finish(P, u, draw, sh.token, sh.mass, lane);
}

}  // namespace

cudaError_t launch_verify_topk(const VerifyParams& p, specdec_dtype dtype, int top_k, cudaStream_t s) {
    const int es = dtype == SPECDEC_BF16 ? 2 : 4;
    const bool vec = ((size_t)p.V * es) % 16 == 0 && reinterpret_cast<uintptr_t>(p.target) % 16 == 0 &&
                     reinterpret_cast<uintptr_t>(p.draft) % 16 == 0;
    const int grid = p.B * (p.K + 1);
    const size_t smem = 2 * CAP * (sizeof(float) + sizeof(int));
    cudaError_t e = cudaSuccess;
#define TK_LAUNCH(TT, VV)                                                                                        \
    do {                                                                                                         \
        e = cudaFuncSetAttribute(verify_topk_kernel<TT, VV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
        if (e == cudaSuccess) verify_topk_kernel<TT, VV><<<grid, TK_THREADS, smem, s>>>(p, top_k);               \
    } while (0)
    if (dtype == SPECDEC_BF16) { if (vec) TK_LAUNCH(__nv_bfloat16, true); else TK_LAUNCH(__nv_bfloat16, false); }
    else { if (vec) TK_LAUNCH(float, true); else TK_LAUNCH(float, false); }
#undef TK_LAUNCH
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}
