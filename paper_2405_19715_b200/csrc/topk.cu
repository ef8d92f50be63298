// Verify/correct under top-k sampling (Appendix D.1 of arXiv 2405.19715: the paper decodes with
// k = 50): both models' logits below the k-th largest of their row count as -inf, then Algorithm 2
// runs on the filtered distributions.
//
// Only about k logits per row matter, so nothing is exponentiated while streaming.  One CTA per
// (row, position); per logit row:
//   1. every thread takes the maximum of its strided share of the row (the one pass that comes
//      from HBM); the smallest, over warps, of each warp's r-th largest thread maximum
//      (r = ceil(k / warps)) is a lower bound on the k-th largest of the row, and a tight one: a
//      share holds 1/512 of the row, so few of the top k collide in one share;
//   2. the pieces of shares (an eighth each) whose maximum reached the bound, about k of 4096, are
//      read again, from L2, and every logit at or above the bound goes into a candidate buffer in
//      shared memory (k plus a few tens);
//   3. the exact k-th largest of the candidates is built bit by bit from counting barriers (each
//      thread holds up to two candidates' order-preserving keys; a radix select takes over when
//      there are more), and the softmax terms of the kept ones are summed.
// The accept test follows, and -- for a rejecting or bonus position -- the residual draw over the
// kept entries: ranked by token id, weights in fp32, prefix in fp64 (the arithmetic of the
// unfiltered kernels).  If the bound turns out too loose for the buffer (rows with -inf or repeated
// maxima), an exact radix select over the row supplies the threshold and the row is filtered again.
#include "verify_device.cuh"

namespace {

using namespace sd;

constexpr int TK_THREADS = 512;
constexpr int TK_WARPS = TK_THREADS / 32;
constexpr int CAP = 4096;                 // candidates per row; every V <= CAP fits whole
constexpr int MAX_KEPT = CAP / 2;         // kept entries (k + ties at the k-th value) the draw can hold

struct TkShared {
    float wrth[TK_WARPS], wmax[TK_WARPS];
    long long zpart[TK_WARPS];
    int count[2], overflow[2];
    float tau[2];
    Norm norm[2];
    unsigned int hist[256];
    unsigned int sel_prefix, sel_rank;
    int state, n_kept, token, retry, nflag;
    float mass;
    unsigned short flist[TK_THREADS * 8];          // (thread, sub-share) pairs that hold a candidate
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

// Pass 1: this thread's maxima over its strided share of the row (NaN ignored).  The share is the
// vectors tid + 512 q; it is kept as SEG sub-shares (q / U mod SEG) so that pass 2 can re-read a
// few vectors instead of the whole share.  Without vector loads the share is one piece (seg[0]).
constexpr int SEG = 8, TM_U = 4;
template <typename T, bool VEC>
__device__ __forceinline__ float thread_max(const T* __restrict__ row, int V, int tid, float (&seg)[SEG]) {
    constexpr int N = Elem<T>::EPV;
#pragma unroll
    for (int s = 0; s < SEG; ++s) seg[s] = -INFINITY;
    if constexpr (VEC) {
        const int nvec = V / N;
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        const uint32_t ninf = neg_inf_word(T());
        for (int base = 0; base < nvec; base += SEG * TM_U * TK_THREADS) {
#pragma unroll
            for (int s = 0; s < SEG; ++s) {
                const int j0 = base + s * TM_U * TK_THREADS + tid;
                if (j0 < nvec) {
                    uint4 r[TM_U];
#pragma unroll
                    for (int k = 0; k < TM_U; ++k) {
                        const int j = j0 + k * TK_THREADS;
                        r[k] = j < nvec ? __ldcg(rv + j) : make_uint4(ninf, ninf, ninf, ninf);
                    }
#pragma unroll
                    for (int k = 0; k < TM_U; ++k) seg[s] = fmaxf(seg[s], vec_max(r[k], T()));
                }
            }
        }
    } else {
        for (int v = tid; v < V; v += TK_THREADS) {
            const float x = to_float(row[v]);
            if (x == x) seg[0] = fmaxf(seg[0], x);
        }
    }
    float m = seg[0];
#pragma unroll
    for (int s = 1; s < SEG; ++s) m = fmaxf(m, seg[s]);
    return m;
}

__device__ __forceinline__ void append(float x, int idx, float* cval, int* cidx, int* count, int* overflow) {
    const int pos = atomicAdd(count, 1);
    if (pos < CAP) { cval[pos] = x; cidx[pos] = idx; }
    else *overflow = 1;
}

// Exclusive prefix of cnt over the warp, the warp's total in `total`.
__device__ __forceinline__ int warp_excl_scan(int cnt, int lane, int& total) {
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    total = __shfl_sync(0xffffffffu, incl, 31);
    return incl - cnt;
}

// Pass 2: every logit at or above the bound goes into the candidate buffer.  Only the sub-shares
// whose maximum reached the bound are read again (from L2): four lanes per flagged sub-share, one
// vector each.  List slots and buffer slots are claimed once per warp.
template <typename T, bool VEC>
__device__ __forceinline__ void filter_row(const T* __restrict__ row, int V, float bound, const float (&seg)[SEG],
                                           float* cval, int* cidx, int* count, int* overflow, TkShared& sh, int tid) {
    constexpr int N = Elem<T>::EPV;
    const int lane = tid & 31, warp = tid >> 5;
    if (tid == 0) sh.nflag = 0;
    __syncthreads();
    {
        unsigned mask = 0;
#pragma unroll
        for (int s = 0; s < (VEC ? SEG : 1); ++s) mask |= (seg[s] >= bound ? 1u : 0u) << s;
        int total, base = 0;
        int pos = warp_excl_scan(__popc(mask), lane, total);
        if (total) {                                   // warp-uniform
            if (lane == 31) base = atomicAdd(&sh.nflag, total);
            pos += __shfl_sync(0xffffffffu, base, 31);
            for (; mask; mask &= mask - 1) sh.flist[pos++] = (unsigned short)(tid | ((__ffs(mask) - 1) << 9));
        }
    }
    __syncthreads();
    const int nflag = sh.nflag;
    if constexpr (VEC) {
        static_assert(32 % TM_U == 0 && TK_THREADS == 512 && SEG <= 8, "entry packing and lane mapping");
        constexpr int EPT = 32 / TM_U;                 // entries a warp reads per trip
        const int nvec = V / N;
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        for (int e0 = warp * EPT; e0 < nflag; e0 += TK_WARPS * EPT) {        // warp-uniform trip count
            const int e = e0 + lane / TM_U;
            int j = nvec;
            if (e < nflag) {
                const int ent = sh.flist[e];
                j = (ent >> 9) * TM_U * TK_THREADS + (ent & 511) + (lane % TM_U) * TK_THREADS;
            }
            while (__any_sync(0xffffffffu, j < nvec)) {
                float x[N];
                unsigned hits = 0;
                if (j < nvec) {
                    const uint4 r = __ldcg(rv + j);
                    unpack(r, x);
#pragma unroll
                    for (int q = 0; q < N; ++q) hits |= (x[q] >= bound && x[q] > -INFINITY ? 1u : 0u) << q;   // masked (-inf) logits are never candidates
                }
                int total, base = 0;
                int pos = warp_excl_scan(__popc(hits), lane, total);
                if (total) {
                    if (lane == 31) base = atomicAdd(count, total);
                    pos += __shfl_sync(0xffffffffu, base, 31);
#pragma unroll
                    for (int q = 0; q < N; ++q)
                        if (hits & (1u << q)) {
                            if (pos < CAP) { cval[pos] = x[q]; cidx[pos] = j * N + q; }
                            else *overflow = 1;
                            ++pos;
                        }
                }
                j += SEG * TM_U * TK_THREADS;
            }
        }
    } else {
        for (int f = warp; f < nflag; f += TK_WARPS)
            for (int v = (int)(sh.flist[f] & 511) + TK_THREADS * lane; v < V; v += TK_THREADS * 32) {
                const float x = to_float(row[v]);
                if (x >= bound && x > -INFINITY) append(x, v, cval, cidx, count, overflow);
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

// Exact k-th largest of n <= 2 * TK_THREADS values in shared memory: the key is built from the top
// bit down, each bit decided by one counting barrier ("are there still k keys at or above this?").
// bf16 data needs only the upper half of the key.  Every thread calls it and gets the result.
template <typename T>
__device__ __forceinline__ float bisect_kth_largest(const float* cv, int n, int k, int tid) {
    const bool h0 = tid < n, h1 = tid + TK_THREADS < n;
    const uint32_t k0 = h0 ? order_key(cv[tid]) : 0u, k1 = h1 ? order_key(cv[tid + TK_THREADS]) : 0u;
    constexpr int LOW = sizeof(T) == 2 ? 16 : 0;
    uint32_t prefix = 0;
    if (n <= TK_THREADS) {
        for (int bit = 31; bit >= LOW; --bit) {
            const uint32_t t = prefix | (1u << bit);
            if (__syncthreads_count(h0 && k0 >= t) >= k) prefix = t;
        }
    } else {
        for (int bit = 31; bit >= LOW; --bit) {
            const uint32_t t = prefix | (1u << bit);
            const int c = __syncthreads_count(h0 && k0 >= t) + __syncthreads_count(h1 && k1 >= t);
            if (c >= k) prefix = t;
        }
    }
    // the low half of a widened bf16's key is all zeros (positive) or all ones (negative)
    if (LOW && !(prefix & 0x80000000u)) prefix |= 0xffffu;
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
    const float c = P.c;

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
        // ---- pass 1: the row's maximum and a lower bound on its k-th largest
        float seg[SEG];
        const float my_max = thread_max<T, VEC>(rows[rr], V, tid, seg);
        const float wr = warp_rth_largest(my_max, rth, lane);
        float wm;
        asm("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(wm) : "f"(my_max));
        if (lane == 0) { sh.wrth[warp] = wr; sh.wmax[warp] = wm; }
        __syncthreads();
        float bound = sh.wrth[0], row_max = sh.wmax[0];
#pragma unroll
        for (int w = 1; w < TK_WARPS; ++w) { bound = fminf(bound, sh.wrth[w]); row_max = fmaxf(row_max, sh.wmax[w]); }
        // ---- pass 2: candidates at or above the bound
        float* cv = cval + rr * CAP;
        int* ci = cidx + rr * CAP;
        filter_row<T, VEC>(rows[rr], V, bound, seg, cv, ci, &sh.count[rr], &sh.overflow[rr], sh, tid);
        __syncthreads();
        if (sh.overflow[rr]) {                         // block-uniform: the bound was too loose
            const T* row = rows[rr];
            const float kth = radix_kth_largest([row](int v) { return to_float(row[v]); }, V, k, sh, tid);
            if (tid == 0) { sh.count[rr] = 0; sh.overflow[rr] = 0; }
            __syncthreads();
            filter_row<T, VEC>(row, V, kth, seg, cv, ci, &sh.count[rr], &sh.overflow[rr], sh, tid);
            __syncthreads();
        }

        // ---- exact k-th largest among the candidates; n <= k: all are kept, tau is their minimum
        const int n = min(sh.count[rr], CAP);
        const int kk = min(k, n);
        float tau = -INFINITY;
        if (n > 2 * TK_THREADS) tau = radix_kth_largest([cv](int q) { return cv[q]; }, n, kk, sh, tid);
        else if (n > 0) tau = bisect_kth_largest<T>(cv, n, kk, tid);

        // ---- softmax terms of the kept candidates against the row maximum (always kept), summed in
        //      fixed point: the candidates sit in the buffer in arrival order, and integer addition
        //      makes the sum independent of it
        const float ref = row_max * c;
        long long z = 0;
        for (int q = tid; q < n; q += TK_THREADS)
            if (cv[q] >= tau) z += (long long)(ex2(fmaf(cv[q], c, -ref)) * 1099511627776.f);       // 2^40
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
        if (lane == 0) sh.zpart[warp] = z;
        __syncthreads();
        if (tid == 0) {
            long long zt = 0;
            for (int w = 0; w < TK_WARPS; ++w) zt += sh.zpart[w];
            const float zs = (float)((double)zt * (1.0 / 1099511627776.0));
            sh.norm[rr] = make_norm(Acc{ref, zs});
            sh.tau[rr] = tau;
        }
    }
    __syncthreads();
    const bool too_many_ties = sh.overflow[0] || (nrows == 2 && sh.overflow[1]);

    // ---- accept test (thread 0)
    const float tau_p = sh.tau[0], tau_q = nrows == 2 ? sh.tau[1] : -INFINITY;
    const Norm np = sh.norm[0], nq = nrows == 2 ? sh.norm[1] : sh.norm[0];
    if (tid == 0) {
        int state = 0;
        if (!u.bonus) {
            float ratio;
            const bool p_in = y_ok && t_y >= tau_p && t_y > -INFINITY, q_in = y_ok && d_y >= tau_q && d_y > -INFINITY;
            if (!p_in) ratio = 0.f;                                      // p'(y) = 0: certain rejection
            else if (!q_in) ratio = INFINITY;
            else ratio = exp2f(fmaf(t_y, c, -np.rs) - fmaf(d_y, c, -nq.rs)) * (np.inv / nq.inv);
            state = (!y_ok || too_many_ties) ? FLAG_BAD : (r_acc >= ratio ? FLAG_REJECT : FLAG_ACCEPT);
            if (!y_ok) atomicOr(P.status, SPECDEC_DATA_BAD_TOKEN);
            if (P.ratio) P.ratio[(size_t)u.b * P.K + u.i] = state == FLAG_BAD ? -1.f : fminf(1.f, ratio);
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
        for (int q = tid; q < n; q += TK_THREADS)
            if (cval[q] >= tau_p) {
                const int pos = atomicAdd(&sh.n_kept, 1);
                if (pos < MAX_KEPT) { ki[pos] = cidx[q]; kv[pos] = cval[q]; }
            }
        __syncthreads();
        const int kept = sh.n_kept;
        if (kept > MAX_KEPT) {                         // thousands of ties at the k-th value
            if (tid == 0) atomicOr(P.status, SPECDEC_DATA_TOPK_TIES);
        } else {
            int* si = cidx;                            // token ids in vocabulary order; the target's candidates are consumed
            int* kr = cidx + CAP / 2;                  // rank of each kept entry
            float* sw = cval;                          // weights in vocabulary order
            const T* drow = rows[1];
            for (int a = warp; a < kept; a += TK_WARPS) {      // position of entry a in vocabulary order
                const int ia = ki[a];
                int rank = 0;
                for (int j = lane; j < kept; j += 32) rank += ki[j] < ia;
                rank = __reduce_add_sync(0xffffffffu, rank);
                if (lane == 0) kr[a] = rank;
            }
            for (int pass = 0; pass < 2; ++pass) {
                const bool resid = !u.bonus && pass == 0;
                __syncthreads();
                for (int a = tid; a < kept; a += TK_THREADS) {
                    const int ia = ki[a];
                    float w = prob(kv[a], c, np);
                    if (resid) {
                        const float dv = to_float(drow[ia]);
                        const float qv = (dv >= tau_q && dv > -INFINITY) ? prob(dv, c, nq) : 0.f;
                        w = fmaxf(w - qv, 0.f);
                    }
                    si[kr[a]] = ia;
                    sw[kr[a]] = w;
                }
                __syncthreads();
                if (warp == 0) {
                    // lane l sums entries [l*seg, (l+1)*seg); a warp scan gives the mass before each segment
                    const int seg = (kept + 31) / 32, a0 = min(lane * seg, kept), a1 = min(a0 + seg, kept);
                    double own = 0.0;
                    for (int a = a0; a < a1; ++a) own += (double)sw[a];
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
                        for (int a = a0; a < a1; ++a) if (sw[a] > 0.f) lastpos = a;
                        if (hit) {
                            if (lane == __ffs(hit) - 1) {
                                double run = incl - own;
                                int tok = -1;
                                for (int a = a0; a < a1; ++a) {
                                    run += (double)sw[a];
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
