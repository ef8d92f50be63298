// Device-side building blocks of verify/correct (Algorithm 2 of arXiv 2405.19715):
// softmax statistics with a lazily re-referenced running sum, the accept test, the
// residual / bonus inverse-CDF draw and the per-row first-rejection ballot.
// Used by the direct kernel (verify.cu) and the streaming kernel (verify_stream.cu).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "specdec_internal.h"

namespace sd {

constexpr float NEG_BIG = -1.0e30f;      // "no reference yet": any finite logit re-references
constexpr int FLAG_ACCEPT = 1, FLAG_REJECT = 2, FLAG_BAD = 3;

// Phase timestamp of a unit, written by the calling thread.  Compiled in only with -DSPECDEC_STAMPS (the
// diagnostic build of the library); the regular build carries no trace of it.
__device__ __forceinline__ void stamp(const VerifyParams& P, int unit, int slot) {
#ifdef SPECDEC_STAMPS
    if (P.stamps) {
        unsigned long long g, c;     // "memory": the reads keep their place between barriers and memory operations
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g)::"memory");
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(c)::"memory");
        unsigned long long* o = P.stamps + ((size_t)unit * SPECDEC_STAMP_SLOTS + slot) * 2;
        o[0] = g;
        o[1] = c;
    }
#endif
}

template <typename T> struct Elem;
template <> struct Elem<float> { static constexpr int EPV = 4; };           // elements per 16 bytes
template <> struct Elem<__nv_bfloat16> { static constexpr int EPV = 8; };

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int32_t* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_relaxed(const int32_t* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed(int32_t* p, int v) {
    asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int atom_add_acq_rel(int32_t* p, int v) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ void unpack(const uint4& r, float (&x)[4]) {
    x[0] = __uint_as_float(r.x); x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z); x[3] = __uint_as_float(r.w);
}
__device__ __forceinline__ void unpack(const uint4& r, float (&x)[8]) {   // 8 bf16 -> fp32, exact
    x[0] = __uint_as_float(r.x << 16); x[1] = __uint_as_float(r.x & 0xffff0000u);
    x[2] = __uint_as_float(r.y << 16); x[3] = __uint_as_float(r.y & 0xffff0000u);
    x[4] = __uint_as_float(r.z << 16); x[5] = __uint_as_float(r.z & 0xffff0000u);
    x[6] = __uint_as_float(r.w << 16); x[7] = __uint_as_float(r.w & 0xffff0000u);
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// Vector j (EPV consecutive elements) of a row.  VEC: one 16-byte load through L2 only.
// Otherwise element loads with everything at or beyond V read as -inf (weight zero).
template <typename T, bool VEC>
__device__ __forceinline__ void load_vec(const T* __restrict__ row, int j, int V, float (&x)[Elem<T>::EPV]) {
    constexpr int N = Elem<T>::EPV;
    if constexpr (VEC) {
        uint4 r = __ldcg(reinterpret_cast<const uint4*>(row) + j);
        unpack(r, x);
    } else {
        const int v0 = j * N;
#pragma unroll
        for (int k = 0; k < N; ++k) x[k] = (v0 + k < V) ? to_float(row[v0 + k]) : -INFINITY;
    }
}

// ---------------------------------------------------------------------------------------
// Running sum of 2^(x*c - rs).  The reference rs follows the data lazily: it is replaced by
// the current vector's maximum only when that vector's terms sum above 256*N, i.e. when some
// logit sits more than ~8 binades above the reference.  Exponent arguments of the terms that
// matter therefore stay small (accurate), nothing can overflow, and the common case costs one
// compare and one not-taken branch per vector instead of a maximum per element.
struct Acc {
    float rs, s;
};
__device__ __forceinline__ Acc acc_init() { return Acc{NEG_BIG, 0.f}; }

template <int N>
__device__ __forceinline__ float sum_tree(const float (&e)[N]) {
    if constexpr (N == 8) return ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
    else return (e[0] + e[1]) + (e[2] + e[3]);
}

template <int N>
__device__ __forceinline__ void acc_update(Acc& a, const float (&x)[N], float c) {
    float e[N];
#pragma unroll
    for (int k = 0; k < N; ++k) e[k] = ex2(fmaf(x[k], c, -a.rs));
    float vs = sum_tree<N>(e);
    if (!(vs <= 256.f * N)) {
        float m = x[0];
#pragma unroll
        for (int k = 1; k < N; ++k) m = fmaxf(m, x[k]);
        if (m >= -3.0e38f) {                       // a finite (or +inf) maximum: re-reference
            const float nrs = m * c;
            a.s *= ex2(a.rs - nrs);
            a.rs = nrs;
#pragma unroll
            for (int k = 0; k < N; ++k) e[k] = ex2(fmaf(x[k], c, -nrs));
            vs = sum_tree<N>(e);
        } else {
            vs = (m != m) ? m : 0.f;               // all NaN propagates; all -inf adds nothing
        }
    }
    a.s += vs;
}

// ---- packed fp32x2 arithmetic ------------------------------------------------------------
using f2 = unsigned long long;
__device__ __forceinline__ f2 pack2(float a, float b) {
    f2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(f2 v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) {
    f2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f2 add2(f2 a, f2 b) {
    f2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f2 mul2(f2 a, f2 b) {
    f2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f2 ex2_2(f2 a) {
    float x, y;
    unpack2(a, x, y);
    return pack2(ex2(x), ex2(y));
}

// Statistics of one row inside a statistics warp: every lane keeps two interleaved partial sums
// of 2^(x*c - rs) against a reference rs that is the same in all lanes of the warp.  Before a
// tile's exponentials are issued the warp takes the maximum of the tile's raw logits (packed
// max, one redux) and moves the reference up if that maximum sits more than 8 binades above it,
// so the hot loop has no data-dependent branch, exponent arguments of the terms that matter
// stay small, and nothing can overflow.
struct Acc2 {
    float rs;
    f2 s;
};
__device__ __forceinline__ Acc2 acc2_init() { return Acc2{NEG_BIG, pack2(0.f, 0.f)}; }
__device__ __forceinline__ Acc acc2_fold(const Acc2& a) {
    float lo, hi;
    unpack2(a.s, lo, hi);
    return Acc{a.rs, lo + hi};
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// Largest element of a 16-byte vector as fp32 (NaNs are skipped).
__device__ __forceinline__ float vec_max(const uint4& r, __nv_bfloat16) {
    const uint32_t m = max_bf16x2(max_bf16x2(r.x, r.y), max_bf16x2(r.z, r.w));
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
}
__device__ __forceinline__ float vec_max(const uint4& r, float) {
    return fmaxf(fmaxf(__uint_as_float(r.x), __uint_as_float(r.y)), fmaxf(__uint_as_float(r.z), __uint_as_float(r.w)));
}
__device__ __forceinline__ uint32_t neg_inf_word(__nv_bfloat16) { return 0xff80ff80u; }
__device__ __forceinline__ uint32_t neg_inf_word(float) { return 0xff800000u; }

// Warp-uniform re-reference: m is this lane's maximum raw logit of the coming tile.
__device__ __forceinline__ void acc2_reference(Acc2& a, float m, float c) {
    float M;
    asm("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(M) : "f"(m));
    const float top = M * c;
    if (top > a.rs + 8.f && M > -3.0e38f) {          // same decision in every lane
        const float f = ex2(a.rs - top);
        a.s = mul2(a.s, pack2(f, f));
        a.rs = top;
    }
}

// The same decision taken by one thread for itself (kernels whose threads keep references of
// their own).
__device__ __forceinline__ void acc2_reference_thread(Acc2& a, float m, float c) {
    const float top = m * c;
    if (top > a.rs + 8.f && m > -3.0e38f) {
        const float f = ex2(a.rs - top);
        a.s = mul2(a.s, pack2(f, f));
        a.rs = top;
    }
}

template <int NP>   // NP packed pairs = 2*NP elements of one 16-byte vector
__device__ __forceinline__ void acc2_add(Acc2& a, const f2 (&x)[NP], f2 c2, f2 nrs) {
    f2 e[NP];
#pragma unroll
    for (int k = 0; k < NP; ++k) e[k] = ex2_2(fma2(x[k], c2, nrs));
    if constexpr (NP == 4) a.s = add2(a.s, add2(add2(e[0], e[1]), add2(e[2], e[3])));
    else a.s = add2(a.s, add2(e[0], e[1]));
}

__device__ __forceinline__ void to_pairs(const uint4& r, f2 (&x)[2], float) {          // 4 fp32
    x[0] = pack2(__uint_as_float(r.x), __uint_as_float(r.y));
    x[1] = pack2(__uint_as_float(r.z), __uint_as_float(r.w));
}
__device__ __forceinline__ void to_pairs(const uint4& r, f2 (&x)[4], __nv_bfloat16) {  // 8 bf16, widened exactly
    x[0] = pack2(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u));
    x[1] = pack2(__uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
    x[2] = pack2(__uint_as_float(r.z << 16), __uint_as_float(r.z & 0xffff0000u));
    x[3] = pack2(__uint_as_float(r.w << 16), __uint_as_float(r.w & 0xffff0000u));
}


__device__ __forceinline__ Acc acc_merge(const Acc& a, const Acc& b) {
    Acc r;
    r.rs = fmaxf(a.rs, b.rs);
    r.s = a.s * ex2(a.rs - r.rs) + b.s * ex2(b.rs - r.rs);
    return r;
}

__device__ __forceinline__ Acc warp_merge(Acc a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Acc b;
        b.rs = __shfl_xor_sync(0xffffffffu, a.rs, o);
        b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
        a = acc_merge(a, b);
    }
    return a;
}

// Normaliser of a row: the reference its terms were summed against and the reciprocal of that sum,
// so that p(x) = 2^(x*c - rs) * inv.  The exponent is formed against the very reference of the
// sum (no common scale error beyond the rounding of one reciprocal) and nothing needs a logarithm.
struct Norm {
    float rs, inv;
};
__device__ __forceinline__ Norm make_norm(const Acc& a) { return Norm{a.rs, 1.f / a.s}; }
__device__ __forceinline__ float prob(float x, float c, const Norm& n) { return ex2(fmaf(x, c, -n.rs)) * n.inv; }

// CTA-wide merge of per-thread statistics, one warp-level step: both rows' references move to the
// warp maximum (one redux each), the rescaled sums are added by a butterfly (identical in every lane).
__device__ __forceinline__ float warp_max(float v) {
    float m;
    asm("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(m) : "f"(v));
    return m;
}
__device__ __forceinline__ void warp_merge2(Acc& p, Acc& q) {
    const float mp = warp_max(p.rs), mq = warp_max(q.rs);
    float sp = p.s * ex2(p.rs - mp), sq = q.s * ex2(q.rs - mq);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sp += __shfl_xor_sync(0xffffffffu, sp, o);
        sq += __shfl_xor_sync(0xffffffffu, sq, o);
    }
    p = Acc{mp, sp};
    q = Acc{mq, sq};
}

// Loads whose place in the instruction stream matters (operands requested early so that their
// latency overlaps the streaming pass): the compiler keeps volatile statements in order.
__device__ __forceinline__ int ld_early_s32(const int32_t* p) {
    int v;
    asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float ld_early_f32(const float* p) {
    float v;
    asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ float ld_early_logit(const float* p) { return ld_early_f32(p); }
__device__ __forceinline__ float ld_early_logit(const __nv_bfloat16* p) {
    unsigned short v;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return __uint_as_float((uint32_t)v << 16);
}

// Scalars fetched into shared memory by asynchronous 4-byte copies.  Unlike a load into a register,
// whose place in the instruction stream the assembler is free to move down to the first use, the
// copy is in flight from the moment it is issued: a scalar asked for before the streaming pass has
// landed long before the pass ends.  scalars_wait() by the issuing thread, then a barrier, make them
// readable by the CTA.
__device__ __forceinline__ void scalar_fetch(uint32_t* smem_dst, const void* gsrc) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
                 : "memory");
}
__device__ __forceinline__ void scalars_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Element e of a row as fp32, fetched as the aligned 4-byte word that holds it (a bf16 element is one
// half of its word).  The word lies inside the tensor whenever the tensor's base is 4-byte aligned.
__device__ __forceinline__ void logit_fetch(uint32_t* smem_dst, const float* row, int e) { scalar_fetch(smem_dst, row + e); }
__device__ __forceinline__ void logit_fetch(uint32_t* smem_dst, const __nv_bfloat16* row, int e) {
    scalar_fetch(smem_dst, reinterpret_cast<const void*>(reinterpret_cast<uintptr_t>(row + e) & ~(uintptr_t)3));
}
__device__ __forceinline__ float logit_fetched(uint32_t w, const float*, int) { return __uint_as_float(w); }
__device__ __forceinline__ float logit_fetched(uint32_t w, const __nv_bfloat16* row, int e) {
    return (reinterpret_cast<uintptr_t>(row + e) & 2) ? __uint_as_float(w & 0xffff0000u) : __uint_as_float(w << 16);
}

// Pass over the two rows of one unit by a CTA of THREADS threads: this thread's share of the
// softmax statistics (merge with warp_merge / acc_merge).  The draft row is skipped at a bonus
// position.  VEC: four vectors of each row in flight per thread; the reference is moved from the
// maximum of the raw inputs, so the exponentials are issued without a data-dependent branch.
struct NoHook {
    __device__ __forceinline__ void operator()() const {}
};
// `after_first_loads` runs once, right after the first round of row loads has been issued and before
// anything waits for it (the place for a dependent scalar load whose latency should hide there).
template <typename T, bool VEC, int THREADS, typename Hook = NoHook>
__device__ __forceinline__ void unit_stats(const T* __restrict__ trow, const T* __restrict__ drow, int V, float c,
                                           bool bonus, int tid, Acc& ap, Acc& aq, Hook after_first_loads = Hook()) {
    constexpr int N = Elem<T>::EPV;
    const int nvec = (V + N - 1) / N;
    if constexpr (VEC) {
        constexpr int U = 4, NP = N / 2;
        const uint4* tv = reinterpret_cast<const uint4*>(trow);
        const uint4* dv = reinterpret_cast<const uint4*>(drow);
        const uint32_t ninf = neg_inf_word(T());
        Acc2 a2 = acc2_init(), q2 = acc2_init();
        for (int j0 = tid; j0 < nvec; j0 += U * THREADS) {
            uint4 rt[U], rd[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = j0 + k * THREADS;
                rt[k] = rd[k] = make_uint4(ninf, ninf, ninf, ninf);
                if (j < nvec) {
                    rt[k] = __ldcg(tv + j);
                    if (!bonus) rd[k] = __ldcg(dv + j);
                }
            }
            if (j0 == tid) after_first_loads();
            float mt = -INFINITY, md = -INFINITY;
#pragma unroll
            for (int k = 0; k < U; ++k) {
                mt = fmaxf(mt, vec_max(rt[k], T()));
                md = fmaxf(md, vec_max(rd[k], T()));
            }
            acc2_reference_thread(a2, mt, c);
            if (!bonus) acc2_reference_thread(q2, md, c);
            const f2 c2 = pack2(c, c);
            const f2 np2 = pack2(-a2.rs, -a2.rs), nq2 = pack2(-q2.rs, -q2.rs);
#pragma unroll
            for (int k = 0; k < U; ++k) {
                f2 xt[NP], xd[NP];
                to_pairs(rt[k], xt, T());
                acc2_add<NP>(a2, xt, c2, np2);
                if (!bonus) {
                    to_pairs(rd[k], xd, T());
                    acc2_add<NP>(q2, xd, c2, nq2);
                }
            }
        }
        if (tid >= nvec) after_first_loads();
        ap = acc2_fold(a2);
        aq = acc2_fold(q2);
    } else {
        after_first_loads();
        float xt[N], xd[N];
        for (int j = tid; j < nvec; j += THREADS) {
            load_vec<T, VEC>(trow, j, V, xt);
            acc_update<N>(ap, xt, c);
            if (!bonus) {
                load_vec<T, VEC>(drow, j, V, xd);
                acc_update<N>(aq, xd, c);
            }
        }
    }
}

// Shared-memory scratch of one CTA handling one (row, position) unit.
struct UnitShared {
    Acc wp[32], wq[32];        // per-warp partial statistics
    Norm np, nq;               // normalisers of the unit
    int need_draw;             // 0 none, 1 residual, 2 target itself
    int token;
    double total;
    uint32_t pre[4];           // scalars fetched ahead: r_i, the words holding t_y and d_y, the uniform of the draw
};

struct Unit {
    int b, i, L;               // row, position, candidate length of the row
    bool bonus;                // i == L: the p_{L+1} row, no draft
};

// p(y) / q(y) from the two base-2 log-probabilities.  p(y) = 0 (a masked target logit) is a certain
// rejection whatever q(y) is -- also when both are zero, where the difference of the logs is not a
// number; q(y) = 0 < p(y) gives +inf (always accepted).
__device__ __forceinline__ float ratio_from_logs(float lp, float lq) {
    const float ratio = exp2f(lp - lq);
    return (lp == -INFINITY || ratio != ratio) ? 0.f : ratio;
}

// Accept test of one unit, called by one full warp once the unit's statistics are known (they
// only need to be valid in lane 0, as do t_y, d_y, y_ok and r = uniforms[b, i]): optional
// outputs and flag publication.  Returns the flag state (0 for the bonus unit) in every lane.
// Flags are plain gpu-scope stores: a flag is self-contained (it carries the call's epoch), and
// the row's arrival counter orders it for the final ballot.
__device__ __forceinline__ int unit_accept(const VerifyParams& P, const Unit& u, const Acc& ap, const Acc& aq,
                                           float t_y, float d_y, int y_ok, float r, int lane, int stamp_unit = -1) {
    const int K = P.K;
    const float LN2 = 0.6931471805599453f;
    int state = 0;
    if (lane == 0) {
        if (!u.bonus) {
            // log2 p(y) and log2 q(y); the references cancel exactly because each term is formed
            // against the same rs the sum was accumulated with.
            const float lp = fmaf(t_y, P.c, -ap.rs) - log2f(ap.s);
            const float lq = fmaf(d_y, P.c, -aq.rs) - log2f(aq.s);
            const float ratio = ratio_from_logs(lp, lq);
            if (stamp_unit >= 0) stamp(P, stamp_unit, 12);
            state = !y_ok ? FLAG_BAD : (r >= ratio ? FLAG_REJECT : FLAG_ACCEPT);   // r == ratio rejects
            if (!y_ok) atomicOr(P.status, SPECDEC_DATA_BAD_TOKEN);
            if (P.ratio) P.ratio[(size_t)u.b * K + u.i] = y_ok ? fminf(1.f, ratio) : -1.f;
            if (P.stats) {
                float4 st;
                st.x = (ap.rs + log2f(ap.s)) * LN2;
                st.y = (aq.rs + log2f(aq.s)) * LN2;
                st.z = exp2f(lp);
                st.w = exp2f(lq);
                reinterpret_cast<float4*>(P.stats)[(size_t)u.b * (K + 1) + u.i] = st;
            }
            st_relaxed(&P.flags[(size_t)u.b * K + u.i], (int)((P.epoch << 2) | (uint32_t)state));
        } else if (P.stats) {
            float4 st = make_float4((ap.rs + log2f(ap.s)) * LN2, 0.f, 0.f, 0.f);
            reinterpret_cast<float4*>(P.stats)[(size_t)u.b * (K + 1) + u.i] = st;
        }
    }
    if (lane == 0 && stamp_unit >= 0) stamp(P, stamp_unit, 13);
    return __shfl_sync(0xffffffffu, state, 0);
}

// Accept test plus the decision whether this unit must produce a draw itself (kernels that draw
// inside the unit): 0 none, 1 from the residual, 2 from the target (bonus position).  A draw is
// needed only if this position can be the first rejection (or is the bonus position); it is
// skipped when an earlier position of the row is already known to have rejected.
__device__ __forceinline__ int unit_decide(const VerifyParams& P, const Unit& u, const Acc& ap, const Acc& aq,
                                           float t_y, float d_y, int y_ok, float r, int lane, int stamp_unit = -1) {
    const int state = unit_accept(P, u, ap, aq, t_y, d_y, y_ok, r, lane, stamp_unit);
    if (!u.bonus && state != FLAG_REJECT) return 0;      // accepted (or bad token): never draws
    bool known = false;
    for (int j0 = 0; j0 < u.i; j0 += 32) {
        const int j = j0 + lane;
        int f = 0;
        if (j < u.i) f = ld_relaxed(&P.flags[(size_t)u.b * P.K + j]);
        known |= __any_sync(0xffffffffu, ((uint32_t)f >> 2) == P.epoch && (f & 3) >= FLAG_REJECT);
    }
    if (known) return 0;
    return u.bonus ? 2 : 1;
}

// Weights y' is drawn from, for one vector: (p - q)_+ (mode 1) or p (mode 2).
template <int N>
__device__ __forceinline__ float vec_weights(const float (&xt)[N], const float (&xd)[N], float c, const Norm& np,
                                             const Norm& nq, int mode, float (&w)[N]) {
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < N; ++k) {
        const float p = prob(xt[k], c, np);
        w[k] = (mode == 1) ? fmaxf(p - prob(xd[k], c, nq), 0.f) : p;
        sum += w[k];
    }
    return sum;
}

// Second half of a draw, run by one full warp once every slab sum is in `slab_sum`: fp64 prefix
// over the slabs and the slab that holds the mass to walk to (draw_find), then a walk inside that
// slab over one vector of weights per lane (draw_walk).
struct SlabPick {
    int slab;                  // the slab that holds tau
    double base;               // mass of the slabs before it
    double tau;                // the mass to walk to
    double total;              // mass of all slabs
};
__device__ __forceinline__ SlabPick draw_find(const float* __restrict__ slab_sum, int nslab, float u01, int lane,
                                              double tau_abs = -1.0) {
    // fp64 prefix over slabs: each lane owns a contiguous run of slabs
    const int per = (nslab + 31) / 32;
    const int s0 = min(lane * per, nslab), s1 = min(s0 + per, nslab);
    double mine = 0.0;
    for (int s = s0; s < s1; ++s) mine += (double)slab_sum[s];
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    SlabPick pk;
    pk.total = __shfl_sync(0xffffffffu, incl, 31);
    // the mass to walk to: u * total, unless the caller fixed it (a draw that spans several CTAs' slices)
    pk.tau = tau_abs >= 0.0 ? tau_abs : (double)u01 * pk.total;
    // first slab whose inclusive prefix exceeds tau
    double run = incl - mine;
    int found = -1;
    double base = 0.0;
    for (int s = s0; s < s1; ++s) {
        const double nxt = run + (double)slab_sum[s];
        if (found < 0 && nxt > pk.tau) { found = s; base = run; }
        run = nxt;
    }
    const unsigned m = __ballot_sync(0xffffffffu, found >= 0);
    if (m) {
        const int src = __ffs(m) - 1;
        pk.slab = __shfl_sync(0xffffffffu, found, src);
        pk.base = __shfl_sync(0xffffffffu, base, src);
    } else {
        // rounding left nothing above tau: take the last slab with positive mass
        int lastpos = -1;
        double lb = 0.0;
        run = incl - mine;
        for (int s = s0; s < s1; ++s) {
            if (slab_sum[s] > 0.f) { lastpos = s; lb = run; }
            run += (double)slab_sum[s];
        }
        const unsigned pm = __ballot_sync(0xffffffffu, lastpos >= 0);
        const int src = pm ? 31 - __clz(pm) : 0;
        pk.slab = __shfl_sync(0xffffffffu, lastpos, src);
        pk.base = __shfl_sync(0xffffffffu, lb, src);
        if (pk.slab < 0) { pk.slab = 0; pk.base = 0.0; }
    }
    return pk;
}

// Walk inside slab pk.slab: lane l holds the N weights w of vector pk.slab * 32 + l (zeros past the row's
// end) and their fp32 sum ls.  Returns the token in every lane.
template <int N>
__device__ __forceinline__ int draw_walk(const SlabPick& pk, const float (&w)[N], float ls, int V, int lane) {
    const int j = pk.slab * 32 + lane;
    float li = ls;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float up = __shfl_up_sync(0xffffffffu, li, o);
        if (lane >= o) li += up;
    }
    float lex = __shfl_up_sync(0xffffffffu, li, 1);
    if (lane == 0) lex = 0.f;
    const unsigned hm = __ballot_sync(0xffffffffu, pk.base + (double)li > pk.tau);
    const unsigned pm = __ballot_sync(0xffffffffu, ls > 0.f);
    const int sel = hm ? __ffs(hm) - 1 : (pm ? 31 - __clz(pm) : -1);
    int tok = min(pk.slab * 32 * N, V - 1);
    if (sel >= 0 && lane == sel) {
        double acc = pk.base + (double)lex;
        int pick = -1, lastp = 0;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            acc += (double)w[k];
            if (w[k] > 0.f) lastp = k;
            if (pick < 0 && acc > pk.tau) pick = k;
        }
        if (pick < 0) pick = lastp;
        tok = min(j * N + pick, V - 1);
    }
    if (sel >= 0) tok = __shfl_sync(0xffffffffu, tok, sel);
    return tok;
}

// draw_find, then the chosen slab's vectors re-read from global memory, then draw_walk.  Returns the
// token; *total_out receives the total mass.
template <typename T, bool VEC>
__device__ __forceinline__ int draw_select(const VerifyParams& P, const T* __restrict__ trow,
                                           const T* __restrict__ drow, int mode, float u01, const Norm np,
                                           const Norm nq, const float* __restrict__ slab_sum, int lane,
                                           double* total_out, double tau_abs = -1.0) {
    constexpr int N = Elem<T>::EPV;
    const int V = P.V;
    const int nvec = (V + N - 1) / N;
    const int nslab = (nvec + 31) / 32;
    const SlabPick pk = draw_find(slab_sum, nslab, u01, lane, tau_abs);
    float xt[N], xd[N], w[N];
#pragma unroll
    for (int k = 0; k < N; ++k) { xd[k] = 0.f; w[k] = 0.f; }
    const int j = pk.slab * 32 + lane;
    float ls = 0.f;
    if (j < nvec) {
        load_vec<T, VEC>(trow, j, V, xt);
        if (mode == 1) load_vec<T, VEC>(drow, j, V, xd);
        ls = vec_weights<N>(xt, xd, P.c, np, nq, mode, w);
    }
    *total_out = pk.total;
    return draw_walk<N>(pk, w, ls, V, lane);
}

// First half of a block-wide draw: the fp32 sum of the weights of every slab of the rows (read from
// global memory, L2) into slab_sum.  A slab is the 32*EPV consecutive elements one warp covers
// with one vector per lane.  All `nthreads` threads (tid 0..nthreads-1, whole warps) must call; the
// caller synchronises before slab_sum is read.
template <typename T, bool VEC>
__device__ __forceinline__ void unit_slabs(const VerifyParams& P, const T* __restrict__ trow,
                                           const T* __restrict__ drow, int mode, const Norm np, const Norm nq,
                                           float* __restrict__ slab_sum, int tid, int nthreads) {
    constexpr int N = Elem<T>::EPV;
    const int V = P.V;
    const int nvec = (V + N - 1) / N;
    const int nslab = (nvec + 31) / 32;
    const int warp = tid >> 5, lane = tid & 31, nwarp = nthreads >> 5;
    float xt[N], xd[N], w[N];
#pragma unroll
    for (int k = 0; k < N; ++k) xd[k] = 0.f;

    if constexpr (VEC) {
        // four slabs per trip: all loads are issued before any of them is consumed
        constexpr int U = 4;
        const uint4* tv = reinterpret_cast<const uint4*>(trow);
        const uint4* dv = reinterpret_cast<const uint4*>(drow);
        for (int s0 = warp; s0 < nslab; s0 += nwarp * U) {
            uint4 rt[U], rd[U];
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int j = (s0 + k * nwarp) * 32 + lane;
                rt[k] = rd[k] = make_uint4(0, 0, 0, 0);
                if (s0 + k * nwarp < nslab && j < nvec) {
                    rt[k] = __ldcg(tv + j);
                    if (mode == 1) rd[k] = __ldcg(dv + j);
                }
            }
#pragma unroll
            for (int k = 0; k < U; ++k) {
                const int s = s0 + k * nwarp;
                if (s >= nslab) break;
                float ls = 0.f;
                if (s * 32 + lane < nvec) {
                    unpack(rt[k], xt);
                    unpack(rd[k], xd);
                    ls = vec_weights<N>(xt, xd, P.c, np, nq, mode, w);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
                if (lane == 0) slab_sum[s] = ls;
            }
        }
    } else {
        for (int s = warp; s < nslab; s += nwarp) {
            const int j = s * 32 + lane;
            float ls = 0.f;
            if (j < nvec) {
                load_vec<T, VEC>(trow, j, V, xt);
                if (mode == 1) load_vec<T, VEC>(drow, j, V, xd);
                ls = vec_weights<N>(xt, xd, P.c, np, nq, mode, w);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
            if (lane == 0) slab_sum[s] = ls;
        }
    }
}

// Total of the slab sums in fp64, by one full warp, added in the order draw_select adds them (so the
// two agree bit for bit).
__device__ __forceinline__ double slab_total(const float* __restrict__ slab_sum, int nslab, int lane) {
    const int per = (nslab + 31) / 32;
    const int s0 = min(lane * per, nslab), s1 = min(s0 + per, nslab);
    double mine = 0.0;
    for (int s = s0; s < s1; ++s) mine += (double)slab_sum[s];
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    return __shfl_sync(0xffffffffu, incl, 31);
}

// Block-wide inverse-CDF draw over the rows of one unit: slab sums in fp32, everything above them
// in fp64.  Leaves the token in sh.token and the total mass in sh.total.  All `nthreads` threads
// (tid 0..nthreads-1, whole warps) must call; uses named barrier `bar_id`.
template <typename T, bool VEC>
__device__ void unit_draw(const VerifyParams& P, const T* __restrict__ trow, const T* __restrict__ drow, int mode,
                          float u01, UnitShared& sh, float* __restrict__ slab_sum, int tid, int nthreads, int bar_id,
                          double tau_abs = -1.0, int stamp_unit = -1) {
    const int warp = tid >> 5, lane = tid & 31;
    const Norm np = sh.np, nq = sh.nq;
    unit_slabs<T, VEC>(P, trow, drow, mode, np, nq, slab_sum, tid, nthreads);
    bar_sync(bar_id, nthreads);
    if (tid == 0 && stamp_unit >= 0) stamp(P, stamp_unit, 6);

    if (warp == 0) {
        double total;
        const int tok = draw_select<T, VEC>(P, trow, drow, mode, u01, np, nq, slab_sum, lane, &total, tau_abs);
        if (lane == 0) { sh.token = tok; sh.total = total; }
    }
    bar_sync(bar_id, nthreads);
}

// Row bookkeeping, by one full warp of a unit.  row_arrive counts the unit on its row and tells
// whether it was the row's last; row_resolve (last arriver only) ballots the accept flags of the
// positions < L into n = first rejection (or L) and reports bad tokens.
__device__ __forceinline__ bool row_arrive(const VerifyParams& P, const Unit& u, int lane) {
    int last = 0;
    // release: this unit's flag (and draw) are visible before the count; acquire: the last
    // arriver sees every other unit's
    if (lane == 0) last = (atom_add_acq_rel(&P.arrive[u.b], 1) == u.L);
    return __shfl_sync(0xffffffffu, last, 0) != 0;
}
__device__ __forceinline__ void row_resolve(const VerifyParams& P, const Unit& u, int lane, int& n, int& bad) {
    n = u.L;
    bad = 0;
    for (int j0 = 0; j0 < u.L; j0 += 32) {
        const int j = j0 + lane;
        int st = FLAG_ACCEPT;
        if (j < u.L) st = ld_acquire(&P.flags[(size_t)u.b * P.K + j]) & 3;
        const unsigned rej = __ballot_sync(0xffffffffu, st >= FLAG_REJECT);
        const unsigned bd = __ballot_sync(0xffffffffu, st == FLAG_BAD);
        if (rej && n == u.L) n = j0 + __ffs(rej) - 1;
        bad |= (bd != 0);
    }
    if (lane == 0) P.arrive[u.b] = 0;               // ready for the next call
    // positions the method never looks at report zeros
    if (P.ratio)
        for (int j = u.L + lane; j < P.K; j += 32) P.ratio[(size_t)u.b * P.K + j] = 0.f;
    if (P.stats)
        for (int j = (u.L + 1) * 4 + lane; j < (P.K + 1) * 4; j += 32) P.stats[(size_t)u.b * (P.K + 1) * 4 + j] = 0.f;
}

// For kernels that draw inside the unit: record the draw, count the arrival, and let the last
// position of the row to arrive pick n and the draw made at position n.
__device__ __forceinline__ void unit_finish(const VerifyParams& P, const Unit& u, int have_draw, int token, float mass,
                                            int lane, int stamp_unit = -1) {
    const int K = P.K;
    if (lane == 0 && have_draw) {
        st_relaxed(&P.draws[(size_t)u.b * (K + 1) + u.i], token);
        st_relaxed(reinterpret_cast<int32_t*>(&P.draw_mass[(size_t)u.b * (K + 1) + u.i]), __float_as_int(mass));
    }
    const bool last = row_arrive(P, u, lane);
    if (lane == 0 && stamp_unit >= 0) stamp(P, stamp_unit, 8);
    if (!last) return;
    int n, bad;
    row_resolve(P, u, lane, n, bad);
    if (lane == 0) {
        int tok = -1;
        float m = 0.f;
        if (!bad) {
            tok = ld_acquire(&P.draws[(size_t)u.b * (K + 1) + n]);
            m = __int_as_float(ld_acquire(reinterpret_cast<const int32_t*>(&P.draw_mass[(size_t)u.b * (K + 1) + n])));
        }
        P.n_acc[u.b] = bad ? -1 : n;
        P.next[u.b] = tok;
        if (P.rmass) P.rmass[u.b] = bad ? 0.f : (n == u.L ? 1.f : m);
    }
}

}  // namespace sd
