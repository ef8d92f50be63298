// Verify/correct (Algorithm 2 of arXiv 2405.19715) in two launches, for batches that fill the machine
// only a few times over.
//
//   verify_split_stats_kernel   The softmax statistics are sums over logit rows, and the rows the method
//                               needs -- target rows 0..L_b and draft rows 0..L_b-1 of every batch row b --
//                               are independent of one another.  The kernel lays them end to end, cuts
//                               each into chunks of 256 threads x 8 vectors (32 KB) and gives every CTA of
//                               a grid that fills the machine exactly once the same number of consecutive
//                               chunks (+-1), whatever the ragged lengths: all CTAs start together, stream
//                               without a barrier across row boundaries, and finish together.  A CTA's
//                               share of a row (a segment) ends as one partial {reference, sum} in global
//                               memory; the CTA that completes a (row, position) unit -- counted per unit,
//                               in chunks -- merges the unit's partials in chunk order, runs the accept test
//                               and stores the accept flag and the normalisers.  No CTA waits for another.
//   verify_split_draw_kernel    One cluster of CTAs per batch row: first rejection n from the row's flags
//                               (warp ballot over the ragged length), then the one draw the row needs --
//                               residual (p_n - q_n)_+ or bonus p_L, Appendix C -- with the vocabulary cut
//                               into one slice per CTA, the slices combined through distributed shared
//                               memory.
//
// The one-CTA-per-unit kernel (verify.cu) keeps a unit's CTA through the accept test, the draw and the row
// bookkeeping; with only a few units per SM those tails, the whole-unit granularity of the last wave and
// the draws of late units decide when the launch ends.
#include <algorithm>

#include "verify_cluster.cuh"

namespace {

using namespace sd;

constexpr int ST_THREADS = 256;                  // four CTAs per SM
constexpr int ST_U = 8;                          // 16-byte vectors in flight per thread
constexpr int ST_CHUNK = ST_THREADS * ST_U;      // vectors per chunk
constexpr int ST_NW = ST_THREADS / 32;
constexpr int DRAW_THREADS = 512, DRAW_NW = DRAW_THREADS / 32;
constexpr int DRAW_U = 4;                        // vectors of each row per thread in the one-round draw

// Chunks [start(g), start(g+1)) of the C chunks belong to CTA g of G: the first C % G CTAs take one more.
struct Partition {
    int q, rem;
    __device__ __forceinline__ int start(int g) const { return g * q + min(g, rem); }
    __device__ __forceinline__ int owner(int c) const {
        const int big = rem * (q + 1);
        return c < big ? c / (q + 1) : rem + (c - big) / q;
    }
};

// Programmatic dependent launch: the second launch may be scheduled while the first drains; it reads
// nothing the first launch writes before this wait, which returns once the first launch has completed.
__device__ __forceinline__ void wait_for_first_launch() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void let_second_launch_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ Acc warp_merge1(Acc a) {          // identical result in every lane
    const float m = warp_max(a.rs);
    float s = a.s * ex2(a.rs - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return Acc{m, s};
}

// Statistics of one logit row from the partials of the CTAs that shared it, merged in chunk order (one
// full warp; `mine` is the calling CTA's own partial, which is not read back from memory).
__device__ __forceinline__ Acc gather_row(const VerifyParams& P, const Partition& part, int row, int cpr, int g_self,
                                          const Acc& mine, int lane) {
    const int g_lo = part.owner(row * cpr), g_hi = part.owner(row * cpr + cpr - 1);
    Acc acc = acc_init();
    for (int g0 = g_lo; g0 <= g_hi; g0 += 32) {
        const int g = g0 + lane;
        Acc v = acc_init();
        if (g <= g_hi && g != g_self) {
            const float2 f = __ldcg(P.partials + row + g);
            v = Acc{f.x, f.y};
        }
        if (g == g_self) v = mine;
        const int n = min(32, g_hi - g0 + 1);
        for (int k = 0; k < n; ++k) {
            Acc o;
            o.rs = __shfl_sync(0xffffffffu, v.rs, k);
            o.s = __shfl_sync(0xffffffffu, v.s, k);
            acc = acc_merge(acc, o);
        }
    }
    return acc;
}

template <typename T>
__global__ void __launch_bounds__(ST_THREADS, 1024 / ST_THREADS) verify_split_stats_kernel(const VerifyParams P, int cpr) {
    constexpr int N = Elem<T>::EPV, NP = N / 2;
    extern __shared__ int smem_i[];
    __shared__ int warp_sum[ST_NW];
    const int B = P.B, K = P.K;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g_self = blockIdx.x;
    // phase timestamps (diagnostic builds), kept at unit index B + CTA: 0 start, 1 lengths summed, 2 segments known,
    // 3 first thread's streaming done, 4 all warps' streaming done, 5 first segment counted, 6 first warp's epilogue done
    const int st_unit = (B + g_self < B * (K + 1)) ? B + g_self : -1;
    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 0);
    int* rowstart = smem_i;                                              // [B + 1] first needed row of every batch row
    int2* seg_info = reinterpret_cast<int2*>(smem_i + ((B + 2) & ~1));    // [nseg] {batch row, row within it}
    // seg_part follows seg_info once the number of segments is known

    // ---- needed rows per batch row (2 L + 1; none for a bad length), exclusive prefix over the batch
    const int per = (B + ST_THREADS - 1) / ST_THREADS;
    const int b0 = min(tid * per, B), b1 = min(b0 + per, B);
    int mine = 0;
    for (int b = b0; b < b1; ++b) {
        const int L = P.lens ? ld_early_s32(P.lens + b) : K;
        const bool ok = (L >= 0 && L <= K);
        if (!ok && g_self == 0) atomicOr(P.status, SPECDEC_DATA_BAD_LENGTH);
        mine += ok ? 2 * L + 1 : 0;
    }
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    int before = 0;
#pragma unroll
    for (int w = 0; w < ST_NW; ++w) before += (w < warp) ? warp_sum[w] : 0;
    int run = before + incl - mine;
    for (int b = b0; b < b1; ++b) {                                      // the lengths again: they are in L1 now
        const int L = P.lens ? P.lens[b] : K;
        rowstart[b] = run;
        run += (L >= 0 && L <= K) ? 2 * L + 1 : 0;
    }
    if (tid == ST_THREADS - 1) rowstart[B] = run;
    __syncthreads();
    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 1);

    // ---- this CTA's chunks and the row segments they cover
    const int C = rowstart[B] * cpr;
    Partition part;
    part.q = C / (int)gridDim.x;
    part.rem = C % (int)gridDim.x;
    const int c0 = part.start(g_self), c1 = part.start(g_self + 1);
    if (c0 >= c1) return;
    const int row_first = c0 / cpr, nseg = (c1 - 1) / cpr - row_first + 1;
    float2* seg_part = reinterpret_cast<float2*>(seg_info + nseg);       // [nseg][ST_NW] per-warp partials
    for (int s = tid; s < nseg; s += ST_THREADS) {
        const int row = row_first + s;
        int lo = 0, hi = B;                                              // largest b with rowstart[b] <= row
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (rowstart[mid] <= row) lo = mid; else hi = mid;
        }
        seg_info[s] = make_int2(lo, row - rowstart[lo]);
    }
    __syncthreads();

    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 2);
    // ---- streaming pass: eight vectors of the current row in flight per thread, no barrier anywhere
    const int nvec = P.V / N;
    const uint32_t ninf = neg_inf_word(T());
    const f2 c2 = pack2(P.c, P.c);
    auto row_ptr = [&](int s) -> const uint4* {
        const int2 si = seg_info[s];
        const int i = si.y >> 1;
        const T* r = (si.y & 1) ? static_cast<const T*>(P.draft) + ((size_t)si.x * K + i) * (size_t)P.V
                                : static_cast<const T*>(P.target) + ((size_t)si.x * (K + 1) + i) * (size_t)P.V;
        return reinterpret_cast<const uint4*>(r);
    };
    auto flush = [&](int s, const Acc2& a2) {
        const Acc m = warp_merge1(acc2_fold(a2));
        if (lane == 0) seg_part[s * ST_NW + warp] = make_float2(m.rs, m.s);
    };
    int seg = 0;
    const uint4* rv = row_ptr(0);
    Acc2 a2 = acc2_init();
    int k = c0 - row_first * cpr;                                        // chunk within the row
    for (int c = c0; c < c1; ++c, ++k) {
        if (k == cpr) {                                                  // next row: close the segment
            flush(seg, a2);
            ++seg;
            k = 0;
            rv = row_ptr(seg);
            a2 = acc2_init();
        }
        const int j0 = k * ST_CHUNK + tid;
        uint4 r[ST_U];
#pragma unroll
        for (int m = 0; m < ST_U; ++m) {
            const int j = j0 + m * ST_THREADS;
            r[m] = make_uint4(ninf, ninf, ninf, ninf);
            if (j < nvec) r[m] = __ldcg(rv + j);
        }
        float mx = -INFINITY;
#pragma unroll
        for (int m = 0; m < ST_U; ++m) mx = fmaxf(mx, vec_max(r[m], T()));
        acc2_reference_thread(a2, mx, P.c);
        const f2 nr2 = pack2(-a2.rs, -a2.rs);
#pragma unroll
        for (int m = 0; m < ST_U; ++m) {
            f2 x[NP];
            to_pairs(r[m], x, T());
            acc2_add<NP>(a2, x, c2, nr2);
        }
    }
    flush(seg, a2);
    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 3);
    let_second_launch_start();
    __syncthreads();
    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 4);

    // ---- one warp per segment: publish the partial, count the chunks on the unit; the CTA that completes
    //      the unit merges its partials and runs the accept test
    for (int s = warp; s < nseg; s += ST_NW) {
        const float2 pw = lane < ST_NW ? seg_part[s * ST_NW + lane] : make_float2(NEG_BIG, 0.f);
        const Acc mine_row = warp_merge1(Acc{pw.x, pw.y});
        const int row = row_first + s;
        const int2 si = seg_info[s];
        Unit u;
        u.b = si.x;
        u.i = si.y >> 1;
        u.L = (rowstart[u.b + 1] - rowstart[u.b] - 1) >> 1;
        u.bonus = (u.i == u.L);
        const int nch = min(c1, (row + 1) * cpr) - max(c0, row * cpr);
        int32_t* counter = P.unit_arrive + (size_t)u.b * (K + 1) + u.i;
        // the scalars of the accept test are requested before the counter's round trip
        int y = 0, last = 0;
        float r_i = 0.f;
        if (lane == 0) {
            if (!u.bonus) {
                y = ld_early_s32(P.tokens + (size_t)u.b * K + u.i);
                r_i = ld_early_f32(P.uniforms + (size_t)u.b * (K + 1) + u.i);
            }
            P.partials[row + g_self] = make_float2(mine_row.rs, mine_row.s);
            // release: the partial is visible before the count; acquire: the last arriver sees the others'
            last = (atom_add_acq_rel(counter, nch) + nch == cpr * (u.bonus ? 1 : 2));
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        __syncwarp();
        if (tid == 0 && st_unit >= 0 && s == 0) stamp(P, st_unit, 5);
        if (!last) continue;
        const size_t V = (size_t)P.V;
        const T* trow = static_cast<const T*>(P.target) + ((size_t)u.b * (K + 1) + u.i) * V;
        const T* drow = u.bonus ? trow : static_cast<const T*>(P.draft) + ((size_t)u.b * K + u.i) * V;
        int y_ok = 1;
        float t_y = 0.f, d_y = 0.f;
        if (lane == 0) {
            *counter = 0;                                                // ready for the next call
            if (!u.bonus) {
                y_ok = (y >= 0 && y < P.V);
                if (y_ok) { t_y = ld_early_logit(trow + y); d_y = ld_early_logit(drow + y); }
            }
        }
        const int row_t = rowstart[u.b] + 2 * u.i;
        const Acc ap = gather_row(P, part, row_t, cpr, row == row_t ? g_self : -1, mine_row, lane);
        const Acc aq = u.bonus ? acc_init() : gather_row(P, part, row_t + 1, cpr, row == row_t + 1 ? g_self : -1, mine_row, lane);
        unit_accept(P, u, ap, aq, t_y, d_y, y_ok, r_i, lane);
        if (lane == 0) {
            const Norm np = make_norm(ap), nq = u.bonus ? np : make_norm(aq);
            P.norms[(size_t)u.b * (K + 1) + u.i] = make_float4(np.rs, np.inv, nq.rs, nq.inv);
        }
    }
    if (tid == 0 && st_unit >= 0) stamp(P, st_unit, 6);
}

// What a draw CTA knows about its batch row after one round of loads: the first rejection n (L when all
// candidates were accepted), whether a drafted token was out of range, and the normalisers at position n.
struct RowState {
    int n, bad;
    Norm np, nq;
};
__device__ __forceinline__ RowState row_state(const VerifyParams& P, int b, int L, int lane) {
    const int K = P.K;
    RowState rs;
    rs.n = L;
    rs.bad = 0;
    float4 nm;
    if (K < 32) {                                 // one lane per position: flags and normalisers together
        int st = FLAG_ACCEPT;
        float4 mine = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane < L) st = __ldcg(P.flags + (size_t)b * K + lane) & 3;
        if (lane <= L) mine = __ldcg(P.norms + (size_t)b * (K + 1) + lane);
        const unsigned rej = __ballot_sync(0xffffffffu, st >= FLAG_REJECT);
        rs.bad = __ballot_sync(0xffffffffu, st == FLAG_BAD) != 0;
        if (rej) rs.n = __ffs(rej) - 1;
        nm.x = __shfl_sync(0xffffffffu, mine.x, rs.n);
        nm.y = __shfl_sync(0xffffffffu, mine.y, rs.n);
        nm.z = __shfl_sync(0xffffffffu, mine.z, rs.n);
        nm.w = __shfl_sync(0xffffffffu, mine.w, rs.n);
    } else {
        for (int j0 = 0; j0 < L; j0 += 32) {
            const int j = j0 + lane;
            int st = FLAG_ACCEPT;
            if (j < L) st = __ldcg(P.flags + (size_t)b * K + j) & 3;
            const unsigned rej = __ballot_sync(0xffffffffu, st >= FLAG_REJECT);
            rs.bad |= __ballot_sync(0xffffffffu, st == FLAG_BAD) != 0;
            if (rej && rs.n == L) rs.n = j0 + __ffs(rej) - 1;
        }
        nm = __ldcg(P.norms + (size_t)b * (K + 1) + rs.n);
    }
    rs.np = Norm{nm.x, nm.y};
    rs.nq = Norm{nm.z, nm.w};
    return rs;
}

// Outputs of a row that has none (bad length, bad token) and the zeros at positions the method never looks at.
__device__ __forceinline__ void row_reports_bad(const VerifyParams& P, int b) {
    P.n_acc[b] = -1;
    P.next[b] = -1;
    if (P.rmass) P.rmass[b] = 0.f;
}
__device__ __forceinline__ void row_zero_fill(const VerifyParams& P, int b, int L, int lane) {
    const int K = P.K;
    if (P.ratio)
        for (int j = L + lane; j < K; j += 32) P.ratio[(size_t)b * K + j] = 0.f;
    if (P.stats)
        for (int j = (L + 1) * 4 + lane; j < (K + 1) * 4; j += 32) P.stats[(size_t)b * (K + 1) * 4 + j] = 0.f;
}

// The draw when a CTA's slice of the row pair is at most DRAW_U vectors per thread and row: one round of
// loads, the vectors stay in registers, and the warp that holds the chosen slab walks it.
template <typename T>
__global__ void __launch_bounds__(DRAW_THREADS, 2) verify_split_draw_kernel(const VerifyParams P, int C, int slice_len) {
    constexpr int N = Elem<T>::EPV;
    __shared__ float slab_sum[DRAW_NW * DRAW_U];
    __shared__ ClusterShared cs;
    __shared__ SlabPick sh_pick;
    __shared__ int sh_owner;
    const uint32_t rank = cl_rank();
    const int b = blockIdx.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = P.K;
    // phase timestamps (diagnostic builds) at unit index b: 0 start, 1 first launch complete, 2 first rejection and
    // normalisers known, 3 slab sums written, 4 slice masses exchanged, 5 row mass known, 6 slab chosen, 7 token stored, 8 end
    const bool st = (rank == 0 && tid == 0);
    if (st) stamp(P, b, 0);
    const int L = P.lens ? ld_early_s32(P.lens + b) : K;
    const float u01 = ld_early_f32(P.uniforms + (size_t)b * (K + 1) + K);
    wait_for_first_launch();
    if (st) stamp(P, b, 1);
    if (L < 0 || L > K) {                        // cluster-uniform; the status bit was set by the first launch
        if (rank == 0 && tid == 0) row_reports_bad(P, b);
        return;
    }
    const RowState rs = row_state(P, b, L, lane);     // every warp for itself: no barrier
    if (rank == 0 && warp == 0) row_zero_fill(P, b, L, lane);
    if (rs.bad) {                                // a drafted token outside the vocabulary: cluster-uniform
        if (rank == 0 && tid == 0) row_reports_bad(P, b);
        return;
    }
    if (st) stamp(P, b, 2);
    const int n = rs.n;
    int mode = (n == L) ? 2 : 1;
    const size_t V = (size_t)P.V;
    const T* trow = static_cast<const T*>(P.target) + ((size_t)b * (K + 1) + n) * V;
    const T* drow = mode == 2 ? trow : static_cast<const T*>(P.draft) + ((size_t)b * K + n) * V;
    const int start = min((int)rank * slice_len, P.V);
    const int len = min(slice_len, P.V - start);
    const int nvec = len / N, nslab = (nvec + 31) / 32;
    const uint4* tv = reinterpret_cast<const uint4*>(trow + start);
    const uint4* dv = reinterpret_cast<const uint4*>(drow + start);

    uint4 rt[DRAW_U], rd[DRAW_U];
#pragma unroll
    for (int k = 0; k < DRAW_U; ++k) {
        const int j = (warp + k * DRAW_NW) * 32 + lane;
        rt[k] = rd[k] = make_uint4(0, 0, 0, 0);
        if (j < nvec) {
            rt[k] = __ldcg(tv + j);
            if (mode == 1) rd[k] = __ldcg(dv + j);
        }
    }
    float xt[N], xd[N], w[N];
    double W_report = 0.0;
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int k = 0; k < DRAW_U; ++k) {
            const int s = warp + k * DRAW_NW;
            float ls = 0.f;
            if (s * 32 + lane < nvec) {
                unpack(rt[k], xt);
                unpack(rd[k], xd);
                ls = vec_weights<N>(xt, xd, P.c, rs.np, rs.nq, mode, w);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
            if (lane == 0 && s < nslab) slab_sum[s] = ls;
        }
        if (st) stamp(P, b, 3);
        __syncthreads();
        if (warp == 0) {
            const double tot = slab_total(slab_sum, nslab, lane);
            if (lane == 0) cs.total = tot;
        }
        cl_sync();                               // every slice's mass is in place
        if (st) stamp(P, b, 4);
        if (warp == 0) {
            const double m = lane < C ? cl_ld_f64(cl_map(&cs.total, lane)) : 0.0;
            double W = 0.0;
            for (int k = 0; k < C; ++k) W += __shfl_sync(0xffffffffu, m, k);
            if (lane == 0) cs.W = W;
        }
        __syncthreads();
        if (st) stamp(P, b, 5);
        if (pass == 0) W_report = cs.W;
        if (pass == 0 && mode == 1 && !(cs.W > 1e-30)) {   // p == q to rounding: draw from p itself (cluster-uniform)
            mode = 2;
            cl_sync();                           // all masses have been read before they are overwritten
            continue;
        }
        break;
    }
    if (warp == 0) {                             // the slice that holds u * W, and inside it the slab
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
        if (owner < 0) {                         // rounding left nothing above u * W: the last slice with mass
            owner = lastpos < 0 ? 0 : lastpos;
            before = 0.0;
            for (int k = 0; k < owner; ++k) before += __shfl_sync(0xffffffffu, m, k);
        }
        if (owner == (int)rank) {
            const double tau = thr - before;
            const SlabPick pk = draw_find(slab_sum, nslab, u01, lane, tau > 0.0 ? tau : 0.0);
            if (lane == 0) sh_pick = pk;
        }
        if (lane == 0) sh_owner = (owner == (int)rank);
    }
    __syncthreads();
    if (st) stamp(P, b, 6);
    if (sh_owner) {
        const SlabPick pk = sh_pick;
        if (warp == pk.slab % DRAW_NW) {         // this warp holds the slab's vectors
            const int kk = pk.slab / DRAW_NW;
            float ls = 0.f;
#pragma unroll
            for (int k = 0; k < N; ++k) w[k] = 0.f;
#pragma unroll
            for (int k = 0; k < DRAW_U; ++k)
                if (k == kk && pk.slab * 32 + lane < nvec) {
                    unpack(rt[k], xt);
                    unpack(rd[k], xd);
                    ls = vec_weights<N>(xt, xd, P.c, rs.np, rs.nq, mode, w);
                }
            const int tok = start + draw_walk<N>(pk, w, ls, len, lane);
            if (lane == 0) {
                P.n_acc[b] = n;
                P.next[b] = tok;
                if (P.rmass) P.rmass[b] = (n == L) ? 1.f : (float)W_report;
                stamp(P, b, 7);
            }
        }
    }
    cl_sync();                                   // nobody leaves while its mass may still be read
    if (st) stamp(P, b, 8);
}

// The same draw for slices of any length (several rounds of loads, the chosen slab read again).
template <typename T>
__global__ void __launch_bounds__(DRAW_THREADS) verify_split_draw_long_kernel(const VerifyParams P, int C, int slice_len) {
    extern __shared__ float slab_sum_dyn[];
    __shared__ ClusterShared cs;
    const uint32_t rank = cl_rank();
    const int b = blockIdx.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = P.K;
    const int L = P.lens ? ld_early_s32(P.lens + b) : K;
    const float u01 = ld_early_f32(P.uniforms + (size_t)b * (K + 1) + K);
    wait_for_first_launch();
    if (L < 0 || L > K) {
        if (rank == 0 && tid == 0) row_reports_bad(P, b);
        return;
    }
    const RowState rs = row_state(P, b, L, lane);
    if (rank == 0 && warp == 0) row_zero_fill(P, b, L, lane);
    if (rs.bad) {
        if (rank == 0 && tid == 0) row_reports_bad(P, b);
        return;
    }
    const int n = rs.n;
    const int mode = (n == L) ? 2 : 1;
    const size_t V = (size_t)P.V;
    const T* trow = static_cast<const T*>(P.target) + ((size_t)b * (K + 1) + n) * V;
    const T* drow = mode == 2 ? trow : static_cast<const T*>(P.draft) + ((size_t)b * K + n) * V;
    const int start = min((int)rank * slice_len, P.V);
    const int len = min(slice_len, P.V - start);
    VerifyParams Ps = P;
    Ps.V = len;
    int tok = -1;
    double W = 0.0;
    if (cluster_draw<T, true, DRAW_THREADS>(Ps, trow + start, drow + start, start, len, mode, u01, rs.np, rs.nq, C, rank,
                                            cs, slab_sum_dyn, &tok, &W)) {
        if (lane == 0) {
            P.n_acc[b] = n;
            P.next[b] = tok;
            if (P.rmass) P.rmass[b] = (n == L) ? 1.f : (float)W;
        }
    }
}

int sm_count_of_current_device() {
    int dev = 0, n = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n;
}

template <typename T>
cudaError_t launch_t(const VerifyParams& p, int sms, cudaStream_t s) {
    constexpr int N = Elem<T>::EPV;
    const int nvec = p.V / N;
    // first launch: a grid that fills the machine once (fewer CTAs than chunks only for the smallest problems)
    const int cpr = (nvec + ST_CHUNK - 1) / ST_CHUNK;
    const long long chunks_max = (long long)p.B * (2 * p.K + 1) * cpr;
    const int grid = (int)std::min<long long>((long long)sms * (1024 / ST_THREADS), chunks_max);
    const int nseg_max = (int)((chunks_max + grid - 1) / grid) / cpr + 2;
    const size_t smem1 = (size_t)((p.B + 2) & ~1) * sizeof(int) + (size_t)nseg_max * (sizeof(int2) + ST_NW * sizeof(float2));
    auto stats = verify_split_stats_kernel<T>;
    cudaError_t e;
    if (smem1 > 40 * 1024) {
        e = cudaFuncSetAttribute(stats, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
        if (e != cudaSuccess) return e;
    }
    stats<<<grid, ST_THREADS, smem1, s>>>(p, cpr);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    // second launch: a cluster per batch row.  Clusters just large enough for a slice to be one round of
    // loads (DRAW_U vectors per thread and row); rows too long for eight such CTAs take the looping kernel.
    int C = 1;
    while (C < CL_MAX && nvec > C * DRAW_THREADS * DRAW_U) C *= 2;
    const bool one_round = nvec <= C * DRAW_THREADS * DRAW_U;
    const int slice_len = cluster_slice_len<T>(p.V, C);
    const size_t smem2 = one_round ? 0 : (size_t)(slice_len / (32 * N)) * sizeof(float);
    auto draw = one_round ? verify_split_draw_kernel<T> : verify_split_draw_long_kernel<T>;
    if (smem2 > 40 * 1024) {
        e = cudaFuncSetAttribute(draw, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * C));
    cfg.blockDim = dim3(DRAW_THREADS);
    cfg.dynamicSmemBytes = smem2;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the first launch drains
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, draw, p, C, slice_len);
}

}  // namespace

// Rows of whole 16-byte vectors on 16-byte boundaries, and a batch whose row prefix fits in shared memory.
bool verify_split_supported(const VerifyParams& p, specdec_dtype dtype) {
    const int n = dtype == SPECDEC_BF16 ? 8 : 4;
    return p.V % n == 0 && reinterpret_cast<uintptr_t>(p.target) % 16 == 0 &&
           reinterpret_cast<uintptr_t>(p.draft) % 16 == 0 && p.B <= 8192 && p.K >= 1;
}

cudaError_t launch_verify_split(const VerifyParams& p, specdec_dtype dtype, int sm_count, cudaStream_t s, int* n_launch) {
    *n_launch = 2;
    const int sms = sm_count > 0 ? sm_count : sm_count_of_current_device();
    return dtype == SPECDEC_BF16 ? launch_t<__nv_bfloat16>(p, sms, s) : launch_t<float>(p, sms, s);
}
