// One (row, position) unit of verify/correct handled by one CTA (Algorithm 2 of arXiv 2405.19715):
// the body shared by the one-CTA-per-unit kernel (verify.cu) and the allocation-free entry point's
// kernel (verify_static.cu), which differ only in where their scratch lives.
#pragma once

#include "verify_device.cuh"

namespace sd {

// The whole unit: scalar operands requested up front, one streaming pass for the softmax statistics of
// both rows, accept test, and -- only where this position may supply y' -- a second pass over the
// same rows for the residual (or bonus) draw; then the row bookkeeping.  `slab_sum` is dynamic shared
// memory of one float per 32-vector slab of a row.
template <typename T, bool VEC, int THREADS>
__device__ __forceinline__ void direct_unit(const VerifyParams& P, float* __restrict__ slab_sum, UnitShared& sh) {
    // position-major unit order: earlier positions of every row are scheduled first, so their
    // accept flags are usually known by the time a later position decides whether to draw
    const int unit = blockIdx.x;
    Unit u;
    u.i = unit / P.B;
    u.b = unit - u.i * P.B;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // phase timestamps (diagnostic builds): 0 start, 1 length known, 2 this thread's pass 1 done, 3 CTA merged,
    // 4 accept test and draw decision, 5 decision seen by the CTA, 6 slab sums, 7 draw done, 8 arrival counted, 9 end
    if (tid == 0) stamp(P, unit, 0);

    // Everything the accept test needs besides the sums.  The length and the drafted token are requested
    // together (their addresses do not depend on the length); once they are known, thread 0 starts
    // asynchronous copies of the uniform of the accept test, of the two logits of the drafted token and
    // of the uniform of the draw into shared memory, and the streaming pass begins: the scalars land
    // while it runs instead of costing dependent round trips after it.
    u.L = P.lens ? ld_early_s32(P.lens + u.b) : P.K;
    int y = 0;
    if (tid == 0 && u.i < P.K) y = ld_early_s32(P.tokens + (size_t)u.b * P.K + u.i);
    // Early exit (optional): the accept flags of the row's earlier positions are asked for in the same round
    // trip.  If one of them already says "rejected" in this call, this position cannot be the first rejection
    // and nothing it could compute can reach the outputs.
    bool earlier_rejected = false;
    if (P.early_exits && warp == 0 && u.i > 0)
        for (int j0 = 0; j0 < u.i; j0 += 32) {
            const int j = j0 + lane;
            const int f = j < u.i ? ld_relaxed(P.flags + (size_t)u.b * P.K + j) : 0;   // other CTAs write these during the launch
            earlier_rejected |= ((uint32_t)f >> 2) == P.epoch && (f & 3) >= FLAG_REJECT;
        }
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
    if (tid == 0) stamp(P, unit, 1);
    if (P.early_exits && u.i > 0) {              // CTA-uniform decision
        if (warp == 0) {
            const bool any = __any_sync(0xffffffffu, earlier_rejected);
            if (lane == 0) sh.need_draw = any;
        }
        __syncthreads();
        const bool leave = sh.need_draw != 0;
        __syncthreads();                         // sh.need_draw is written again below
        if (leave) {
            if (warp == 0) {
                if (lane == 0) {                 // the drafted token is still range-checked; the flag is this call's
                    const bool y_bad = !u.bonus && (y < 0 || y >= P.V);
                    if (y_bad) atomicOr(P.status, SPECDEC_DATA_BAD_TOKEN);
                    if (!u.bonus) st_relaxed(&P.flags[(size_t)u.b * P.K + u.i], (int)((P.epoch << 2) | (uint32_t)(y_bad ? FLAG_BAD : 0)));
                    atomicAdd(P.early_exits, u.bonus ? 1ull : 2ull);      // logit rows this unit did not read
                }
                unit_finish(P, u, 0, -1, 0.f, lane, unit);
            }
            return;
        }
    }

    const size_t V = (size_t)P.V;
    const T* trow = static_cast<const T*>(P.target) + ((size_t)u.b * (P.K + 1) + u.i) * V;
    const T* drow = u.bonus ? trow : static_cast<const T*>(P.draft) + ((size_t)u.b * P.K + u.i) * V;

    int y_ok = 1;
    if (tid == 0) {
        const float* ur = P.uniforms + (size_t)u.b * (P.K + 1);
        scalar_fetch(&sh.pre[3], ur + P.K);
        if (!u.bonus) {
            scalar_fetch(&sh.pre[0], ur + u.i);
            y_ok = (y >= 0 && y < P.V);
            if (y_ok) { logit_fetch(&sh.pre[1], trow, y); logit_fetch(&sh.pre[2], drow, y); }
        }
        stamp(P, unit, 10);                      // scalars requested
    }

    // ---- pass 1: softmax statistics of both rows
    Acc ap = acc_init(), aq = acc_init();
    unit_stats<T, VEC, THREADS>(trow, drow, P.V, P.c, u.bonus, tid, ap, aq);
    if (tid == 0) { stamp(P, unit, 2); scalars_wait(); }
    if (lane == 0 && warp < 16) stamp(P, unit, 16 + warp);
    warp_merge2(ap, aq);
    if (lane == 0) { sh.wp[warp] = ap; sh.wq[warp] = aq; }
    __syncthreads();
    if (tid == 0) stamp(P, unit, 3);
    if (warp == 0) {
        constexpr int NW = THREADS / 32;
        Acc a = lane < NW ? sh.wp[lane] : acc_init(), b = lane < NW ? sh.wq[lane] : acc_init();
        warp_merge2(a, b);
        if (lane == 0) stamp(P, unit, 11);
        const float r = __uint_as_float(sh.pre[0]);
        const float t_y = logit_fetched(sh.pre[1], trow, y), d_y = logit_fetched(sh.pre[2], drow, y);
        const int mode = unit_decide(P, u, a, b, t_y, d_y, y_ok, r, lane, unit);
        if (lane == 0) {
            sh.np = make_norm(a);
            sh.nq = u.bonus ? sh.np : make_norm(b);
            sh.need_draw = mode;
            stamp(P, unit, 4);
        }
    }
    __syncthreads();
    if (tid == 0) stamp(P, unit, 5);

    // ---- pass 2 (only where this position may supply y'): weights, prefix, inverse CDF
    const int mode = sh.need_draw;
    if (mode) {
        const float u01 = __uint_as_float(sh.pre[3]);
        unit_draw<T, VEC>(P, trow, drow, mode, u01, sh, slab_sum, tid, THREADS, 0, -1.0, unit);
        if (mode == 1 && !(sh.total > 1e-30)) {   // p == q to rounding: draw from p itself
            const double keep = sh.total;
            __syncthreads();
            unit_draw<T, VEC>(P, trow, drow, 2, u01, sh, slab_sum, tid, THREADS, 0);
            if (tid == 0) sh.total = keep;
            __syncthreads();
        }
    }
    if (tid == 0) stamp(P, unit, 7);
    if (warp == 0) unit_finish(P, u, mode != 0, sh.token, mode ? (float)sh.total : 0.f, lane, unit);
    if (tid == 0) stamp(P, unit, 9);
}

}  // namespace sd
