// Streaming verify/correct kernels (Algorithm 2 of arXiv 2405.19715; see specdec.h).
//
// Two launches of persistent CTAs (one per SM) that share one pipeline shape: a producer warp
// moves logit rows from HBM into a shared-memory ring with 1-D bulk async copies (TMA,
// completion on mbarriers), worker warps consume the tiles, and epilogue warps finish each
// unit off the streaming path.
//
//   1. verify_stream_stats_kernel streams every needed (row, position) unit once.  Worker warps
//      form the softmax partial sums (one ex2 per element, packed fp32x2 arithmetic, no
//      data-dependent branch); at the end of a unit they post their partials to a hand-off slot
//      and go straight on.  Epilogue warps merge them, run the accept test, publish the flag and
//      the normalisers, count the unit on its row; the row's last unit ballots the flags into n
//      and queues the row's one draw (b, n).
//   2. verify_stream_draw_kernel streams the two rows of each queued draw again (B units, about
//      1/(K+1) of the first launch's bytes, largely L2 hits), worker warps form the residual (or
//      target) weights and their 256-element slab sums, an epilogue warp picks the token.
//
// The long chain of dependent global accesses of an epilogue (tokens, flags, counters) therefore
// never stalls the stream, and the one draw a row needs is itself a bandwidth-shaped job.
#include "verify_device.cuh"

namespace {

using namespace sd;

#ifndef SPECDEC_STREAM_NS
#define SPECDEC_STREAM_NS 16
#endif
#ifndef SPECDEC_STREAM_TILE
#define SPECDEC_STREAM_TILE 32768
#endif
#ifndef SPECDEC_STREAM_STAGES
#define SPECDEC_STREAM_STAGES 3
#endif
#ifndef SPECDEC_STREAM_NE
#define SPECDEC_STREAM_NE 4
#endif
constexpr int NS = SPECDEC_STREAM_NS;           // statistics warps (consume the ring)
constexpr int NST = NS * 32;
constexpr int NE = SPECDEC_STREAM_NE;           // epilogue warps (accept test, draw, row bookkeeping)
constexpr int STREAM_THREADS = (NS + 1 + NE) * 32;   // + one producer warp
constexpr int TILE_BYTES = SPECDEC_STREAM_TILE; // bytes of one row per ring stage
constexpr int STAGES = SPECDEC_STREAM_STAGES;
constexpr int RING_BYTES = STAGES * 2 * TILE_BYTES;
constexpr int QSLOTS = 16;                      // hand-off slots between statistics and epilogue warps
constexpr int MAX_CAND = 2048;                  // candidate units per CTA whose length is cached
constexpr uint32_t WAIT_POLLS = 1u << 24;       // bound on every mbarrier wait
constexpr int ITERS = TILE_BYTES / 16 / NST;    // 16-byte vectors of one row tile per statistics thread
static_assert(NS <= 32, "one lane of an epilogue warp per statistics warp");
static_assert(ITERS * NST * 16 == TILE_BYTES && ITERS >= 1, "tile must split evenly over the statistics threads");

struct StreamShared {
    unsigned long long full[STAGES];            // ring stage filled by the producer's copies
    unsigned long long empty[STAGES];           // ring stage drained by all worker warps
    unsigned long long slot_full[QSLOTS];       // every worker warp has posted its results of a unit
    unsigned long long slot_empty[QSLOTS];      // an epilogue warp has read them
    unsigned int next_seq;                      // next unit (per-CTA sequence number) without an epilogue warp
    float4 slots[QSLOTS][NS];                   // stats kernel, per worker warp: {rs_p, s_p, rs_q, s_q}
    int cand_L[MAX_CAND];                       // stats kernel: cand_len of this CTA's k-th candidate unit
};

// ---- PTX wrappers -----------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  A wait that runs out records SPECDEC_DATA_WAIT_LIMIT and returns; control flow
// never depends on it, so no thread can be left behind at a barrier (outputs are then invalid).
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, uint32_t* status) {
    for (uint32_t it = 0; it < WAIT_POLLS; ++it)
        if (mbar_try_wait(bar, parity)) return;
    atomicOr(status, SPECDEC_DATA_WAIT_LIMIT);
}
// Warp-wide wait in which only lane 0 spins (the other lanes test once, after it has succeeded),
// so that waiting warps do not flood the shared-memory pipe the working warps read through.
__device__ __forceinline__ void mbar_wait_warp(uint32_t bar, uint32_t parity, uint32_t* status, int lane) {
    if (lane == 0) mbar_wait(bar, parity, status);
    __syncwarp();
    if (lane != 0) mbar_wait(bar, parity, status);
}
// Patient wait for warps that are off the critical path: sleeps between polls.
__device__ __forceinline__ void mbar_wait_relaxed(uint32_t bar, uint32_t parity, uint32_t* status, int lane) {
    if (lane == 0) {
        bool ok = false;
        for (uint32_t it = 0; it < WAIT_POLLS && !(ok = mbar_try_wait(bar, parity)); ++it) __nanosleep(256);
        if (!ok) atomicOr(status, SPECDEC_DATA_WAIT_LIMIT);
    }
    __syncwarp();
    if (lane != 0) mbar_wait(bar, parity, status);
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

// Unit walk shared by all roles: the next live unit at or after candidate k of this CTA
// (candidate k is unit blockIdx.x + k * gridDim.x in position-major order).  The candidate
// lengths were gathered into shared memory once at kernel start (cand_L[k] = cand_len of the
// candidate's row), so the walk costs no global round trip.  Rows with a bad length are reported
// once (by the caller that passes report = true) and skipped; positions beyond L are skipped.
__device__ __forceinline__ bool next_unit(const VerifyParams& P, const int* cand_L, int& k, int ncand, Unit& out,
                                          bool report) {
    for (; k < ncand; ++k) {
        const int u = blockIdx.x + k * gridDim.x;
        const int i = u / P.B, b = u - i * P.B;
        const int L = k < MAX_CAND ? cand_L[k] : (P.lens ? P.lens[b] : P.K);
        if (L < 0 || L > P.K) {
            if (report && i == 0) {
                atomicOr(P.status, SPECDEC_DATA_BAD_LENGTH);
                P.n_acc[b] = -1;
                P.next[b] = -1;
                if (P.rmass) P.rmass[b] = 0.f;
            }
            continue;
        }
        if (i > L) continue;
        out.b = b; out.i = i; out.L = L; out.bonus = (i == L);
        return true;
    }
    return false;
}

__device__ __forceinline__ void stream_init(StreamShared& ss, int tid) {
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ss.full[s]), 1);
            mbar_init(smem_u32(&ss.empty[s]), NS);
        }
        for (int s = 0; s < QSLOTS; ++s) {
            mbar_init(smem_u32(&ss.slot_full[s]), NS);
            mbar_init(smem_u32(&ss.slot_empty[s]), 1);
        }
        ss.next_seq = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
}

// Producer side of one unit: stream `ntiles` tiles of the target row (and the draft row unless
// `single`) into the ring.
__device__ __forceinline__ void produce_unit(StreamShared& ss, uint32_t ring, const unsigned char* tsrc,
                                             const unsigned char* dsrc, bool single, uint32_t row_bytes, int ntiles,
                                             uint32_t& stage, uint32_t& phase, uint32_t* status) {
    for (int t = 0; t < ntiles; ++t) {
        const uint32_t off = (uint32_t)t * TILE_BYTES;
        const uint32_t bytes = min((uint32_t)TILE_BYTES, row_bytes - off);
        const uint32_t full = smem_u32(&ss.full[stage]);
        mbar_wait(smem_u32(&ss.empty[stage]), phase ^ 1u, status);
        mbar_expect_tx(full, single ? bytes : 2 * bytes);
        const uint32_t dst = ring + stage * (2 * TILE_BYTES);
        bulk_load(dst, tsrc + off, bytes, full);
        if (!single) bulk_load(dst + TILE_BYTES, dsrc + off, bytes, full);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
    }
}

// The statistics warps' walk over the CTA's units: every thread keeps the vectors of a tile in registers,
// the warp-uniform reference follows the tile maxima, and at the end of a unit each warp posts its partial
// {reference, sum} of both rows into a hand-off slot for the epilogue warps.  `stage` / `phase` are the
// warp's place in the ring and stay valid for whatever the caller streams next.
template <typename T>
__device__ __forceinline__ void stats_workers(const VerifyParams& P, StreamShared& ss, uint32_t ring, uint32_t row_bytes,
                                              int ntiles, int ncand, int tid, int lane, int warp, uint32_t& stage,
                                              uint32_t& phase) {
    constexpr int NP = Elem<T>::EPV / 2;
    int k = 0;
    Unit un;
    uint32_t seq = 0;
    while (next_unit(P, ss.cand_L, k, ncand, un, false)) {
        Acc2 ap = acc2_init(), aq = acc2_init();
        for (int t = 0; t < ntiles; ++t) {
            const uint32_t bytes = min((uint32_t)TILE_BYTES, row_bytes - (uint32_t)t * TILE_BYTES);
            const int nvec = bytes >> 4;
            const uint32_t base = ring + stage * (2 * TILE_BYTES);
            mbar_wait_warp(smem_u32(&ss.full[stage]), phase, P.status, lane);
            // the tile's vectors of this thread, padded with -inf beyond the row's end
            uint4 rt[ITERS], rd[ITERS];
            float mt = -INFINITY, md = -INFINITY;
#pragma unroll
            for (int j = 0; j < ITERS; ++j) {
                const int v = tid + j * NST;
                const uint32_t ninf = neg_inf_word(T());
                rt[j] = rd[j] = make_uint4(ninf, ninf, ninf, ninf);
                if (v < nvec) {
                    rt[j] = lds128(base + v * 16);
                    if (!un.bonus) rd[j] = lds128(base + TILE_BYTES + v * 16);
                }
                mt = fmaxf(mt, vec_max(rt[j], T()));
                md = fmaxf(md, vec_max(rd[j], T()));
            }
            acc2_reference(ap, mt, P.c);
            if (!un.bonus) acc2_reference(aq, md, P.c);
            const f2 c2 = pack2(P.c, P.c);
            const f2 np2 = pack2(-ap.rs, -ap.rs), nq2 = pack2(-aq.rs, -aq.rs);
#pragma unroll
            for (int j = 0; j < ITERS; ++j) {
                f2 xt[NP], xd[NP];
                to_pairs(rt[j], xt, T());
                acc2_add<NP>(ap, xt, c2, np2);
                if (!un.bonus) {
                    to_pairs(rd[j], xd, T());
                    acc2_add<NP>(aq, xd, c2, nq2);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ss.empty[stage]));
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        // hand the unit's partial sums to the epilogue warps and move on
        Acc fp = acc2_fold(ap), fq = acc2_fold(aq);      // rs is warp-uniform: add the lanes
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            fp.s += __shfl_xor_sync(0xffffffffu, fp.s, o);
            fq.s += __shfl_xor_sync(0xffffffffu, fq.s, o);
        }
        const uint32_t slot = seq % QSLOTS, use = seq / QSLOTS;
        if (lane == 0) {
            if (use > 0) mbar_wait(smem_u32(&ss.slot_empty[slot]), (use - 1) & 1u, P.status);
            ss.slots[slot][warp] = make_float4(fp.rs, fp.s, fq.rs, fq.s);
            mbar_arrive(smem_u32(&ss.slot_full[slot]));
        }
        ++seq;
        ++k;
    }
}

template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1) verify_stream_stats_kernel(const VerifyParams P) {
    extern __shared__ __align__(1024) unsigned char smem[];
    StreamShared& ss = *reinterpret_cast<StreamShared*>(smem + RING_BYTES);
    const uint32_t ring = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    stream_init(ss, tid);
    const int total = (P.K + 1) * P.B;
    const int ncand = (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    for (int k = tid; k < min(ncand, MAX_CAND); k += STREAM_THREADS) {
        const int u = blockIdx.x + k * gridDim.x;
        ss.cand_L[k] = P.lens ? P.lens[u % P.B] : P.K;
    }
    __syncthreads();

    const uint32_t row_bytes = (uint32_t)P.V * sizeof(T);
    const int ntiles = (row_bytes + TILE_BYTES - 1) / TILE_BYTES;
    int k = 0;                      // candidate index of the walk
    Unit un;

    if (warp == NS) {
        // ------------------------------------------------------------------ producer
        if (lane != 0) return;
        const unsigned char* tbase = static_cast<const unsigned char*>(P.target);
        const unsigned char* dbase = static_cast<const unsigned char*>(P.draft);
        uint32_t stage = 0, phase = 0;
        while (next_unit(P, ss.cand_L, k, ncand, un, false)) {
            produce_unit(ss, ring, tbase + ((size_t)un.b * (P.K + 1) + un.i) * row_bytes,
                         dbase + ((size_t)un.b * P.K + un.i) * row_bytes, un.bonus, row_bytes, ntiles, stage, phase,
                         P.status);
            ++k;
        }
        return;   // every copy it issued is awaited by the worker warps before they exit
    }

    if (warp < NS) {
        // ------------------------------------------------------------------ worker warps
        uint32_t stage = 0, phase = 0;
        stats_workers<T>(P, ss, ring, row_bytes, ntiles, ncand, tid, lane, warp, stage, phase);
        return;
    }

    // ------------------------------------------------------------------ epilogue warps
    // Each takes the next unit nobody has claimed yet.
    uint32_t walked = 0;            // sequence number of the unit `un` describes
    bool have = next_unit(P, ss.cand_L, k, ncand, un, lane == 0);
    for (;;) {
        uint32_t seq = 0;
        if (lane == 0) seq = atomicAdd(&ss.next_seq, 1u);
        seq = __shfl_sync(0xffffffffu, seq, 0);
        while (have && walked < seq) {
            ++k;
            have = next_unit(P, ss.cand_L, k, ncand, un, lane == 0);
            ++walked;
        }
        if (!have) break;
        const T* trow = static_cast<const T*>(P.target) + ((size_t)un.b * (P.K + 1) + un.i) * (size_t)P.V;
        const T* drow = un.bonus ? trow : static_cast<const T*>(P.draft) + ((size_t)un.b * P.K + un.i) * (size_t)P.V;
        // everything the accept test needs besides the sums is fetched while the rows stream in
        int y_ok = 1;
        float t_y = 0.f, d_y = 0.f, r = 0.f;
        if (lane == 0 && !un.bonus) {
            r = P.uniforms[(size_t)un.b * (P.K + 1) + un.i];
            const int y = P.tokens[(size_t)un.b * P.K + un.i];
            y_ok = (y >= 0 && y < P.V);
            if (y_ok) { t_y = to_float(trow[y]); d_y = to_float(drow[y]); }
        }
        const uint32_t slot = seq % QSLOTS, use = seq / QSLOTS;
        mbar_wait_relaxed(smem_u32(&ss.slot_full[slot]), use & 1u, P.status, lane);
        Acc a = acc_init(), b = acc_init();
        if (lane < NS) {
            const float4 v = ss.slots[slot][lane];
            a = Acc{v.x, v.y};
            b = Acc{v.z, v.w};
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ss.slot_empty[slot]));
        a = warp_merge(a);
        b = warp_merge(b);
        if (lane == 0) {
            const Norm np = make_norm(a), nq = un.bonus ? np : make_norm(b);
            P.norms[(size_t)un.b * (P.K + 1) + un.i] = make_float4(np.rs, np.inv, nq.rs, nq.inv);
        }
        unit_accept(P, un, a, b, t_y, d_y, y_ok, r, lane);
        if (!row_arrive(P, un, lane)) continue;
        // last unit of its row: first rejection, then queue the row's one draw
        int n, bad;
        row_resolve(P, un, lane, n, bad);
        if (lane == 0) {
            P.n_acc[un.b] = bad ? -1 : n;
            if (bad) {
                P.next[un.b] = -1;
                if (P.rmass) P.rmass[un.b] = 0.f;
            } else {
                P.tasks[atomicAdd(&P.task_ctl[0], 1)] = make_int2(un.b, n);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Draw kernel: task t = (b, n) of the queue; weights w = (p_n - q_n)_+ if n < L else p_L.
template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1) verify_stream_draw_kernel(const VerifyParams P) {
    constexpr int N = Elem<T>::EPV;
    extern __shared__ __align__(1024) unsigned char smem[];
    StreamShared& ss = *reinterpret_cast<StreamShared*>(smem + RING_BYTES);
    const int nvec_row = (P.V + N - 1) / N;
    const int nslab = (nvec_row + 31) / 32;
    float* slab_base = reinterpret_cast<float*>(smem + RING_BYTES + sizeof(StreamShared));   // [QSLOTS_DRAW][nslab]
    constexpr int QD = 2;           // slab-sum buffers in flight between workers and epilogue
    const uint32_t ring = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    stream_init(ss, tid);
    __syncthreads();

    const int ntask = *reinterpret_cast<volatile int*>(&P.task_ctl[0]);
    const uint32_t row_bytes = (uint32_t)P.V * sizeof(T);
    const int ntiles = (row_bytes + TILE_BYTES - 1) / TILE_BYTES;

    if (warp == NS) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const unsigned char* tbase = static_cast<const unsigned char*>(P.target);
            const unsigned char* dbase = static_cast<const unsigned char*>(P.draft);
            uint32_t stage = 0, phase = 0;
            for (int t = blockIdx.x; t < ntask; t += gridDim.x) {
                const int2 task = P.tasks[t];
                const int L = P.lens ? P.lens[task.x] : P.K;
                produce_unit(ss, ring, tbase + ((size_t)task.x * (P.K + 1) + task.y) * row_bytes,
                             dbase + ((size_t)task.x * P.K + task.y) * row_bytes, task.y >= L, row_bytes, ntiles,
                             stage, phase, P.status);
            }
        }
    } else if (warp < NS) {
        // ------------------------------------------------------------------ worker warps
        uint32_t stage = 0, phase = 0, seq = 0;
        for (int t = blockIdx.x; t < ntask; t += gridDim.x, ++seq) {
            const int2 task = P.tasks[t];
            const int L = P.lens ? P.lens[task.x] : P.K;
            const int mode = task.y >= L ? 2 : 1;
            const float4 nv = P.norms[(size_t)task.x * (P.K + 1) + task.y];
            const Norm np{nv.x, nv.y}, nq{nv.z, nv.w};
            const uint32_t slot = seq % QD, use = seq / QD;
            float* slab_sum = slab_base + (size_t)slot * nslab;
            if (use > 0) mbar_wait_warp(smem_u32(&ss.slot_empty[slot]), (use - 1) & 1u, P.status, lane);
            for (int tl = 0; tl < ntiles; ++tl) {
                const uint32_t bytes = min((uint32_t)TILE_BYTES, row_bytes - (uint32_t)tl * TILE_BYTES);
                const int nvec = bytes >> 4;
                const uint32_t base = ring + stage * (2 * TILE_BYTES);
                mbar_wait_warp(smem_u32(&ss.full[stage]), phase, P.status, lane);
#pragma unroll
                for (int j = 0; j < ITERS; ++j) {
                    const int v = tid + j * NST;         // vector of the tile; warp-aligned, so one slab per warp
                    float ls = 0.f;
                    if (v < nvec) {
                        float xt[N], xd[N], w[N];
                        unpack(lds128(base + v * 16), xt);
                        if (mode == 1) unpack(lds128(base + TILE_BYTES + v * 16), xd);
                        else {
#pragma unroll
                            for (int q = 0; q < N; ++q) xd[q] = 0.f;
                        }
                        ls = vec_weights<N>(xt, xd, P.c, np, nq, mode, w);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
                    const int slab = tl * (TILE_BYTES / 16 / 32) + j * NS + warp;
                    if (lane == 0 && slab < nslab) slab_sum[slab] = ls;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ss.empty[stage]));
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (lane == 0) mbar_arrive(smem_u32(&ss.slot_full[slot]));
        }
    } else if (warp == NS + 1) {
        // ------------------------------------------------------------------ epilogue warp
        uint32_t seq = 0;
        for (int t = blockIdx.x; t < ntask; t += gridDim.x, ++seq) {
            const int2 task = P.tasks[t];
            const int b = task.x, n = task.y;
            const int L = P.lens ? P.lens[b] : P.K;
            int mode = n >= L ? 2 : 1;
            const float4 nv = P.norms[(size_t)b * (P.K + 1) + n];
            const Norm np{nv.x, nv.y}, nq{nv.z, nv.w};
            const float u01 = P.uniforms[(size_t)b * (P.K + 1) + P.K];
            const T* trow = static_cast<const T*>(P.target) + ((size_t)b * (P.K + 1) + n) * (size_t)P.V;
            const T* drow = mode == 2 ? trow : static_cast<const T*>(P.draft) + ((size_t)b * P.K + n) * (size_t)P.V;
            const uint32_t slot = seq % QD, use = seq / QD;
            float* slab_sum = slab_base + (size_t)slot * nslab;
            mbar_wait_relaxed(smem_u32(&ss.slot_full[slot]), use & 1u, P.status, lane);
            double total;
            int tok = draw_select<T, true>(P, trow, drow, mode, u01, np, nq, slab_sum, lane, &total);
            const double mass = total;
            if (mode == 1 && !(total > 1e-30)) {
                // p == q to rounding: draw from p itself (rare; this warp re-forms the slab sums alone)
                __shared__ UnitShared fallback_sh;
                if (lane == 0) { fallback_sh.np = np; fallback_sh.nq = nq; }
                __syncwarp();
                unit_draw<T, true>(P, trow, drow, 2, u01, fallback_sh, slab_sum, lane, 32, 2);
                tok = fallback_sh.token;
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ss.slot_empty[slot]));
                P.next[b] = tok;
                if (P.rmass) P.rmass[b] = n >= L ? 1.f : (float)mass;
            }
        }
    }
    // the last CTA to finish empties the queue for the next call
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(&P.task_ctl[1], 1) == (int)gridDim.x - 1) {
            P.task_ctl[0] = 0;
            P.task_ctl[1] = 0;
        }
    }
}

// =============================================================================================
// Fused kernel: the same pipeline in one launch.  Phase 1 is the statistics pass above.  Every row
// of the batch ends in exactly one record, a single word {epoch, mode, n} stored (release) by the
// epilogue warp that resolves the row (mode 0 for rows that draw nothing: bad length or bad
// token).  When a CTA's producer has streamed its last unit it claims rows in order (head++),
// waits (bounded) for the row's record, fetches the row's normalisers and uniform, and streams
// that row pair through the same ring as a draw unit, described to the
// worker and epilogue warps by a small descriptor ring in shared memory; a claim >= B ends the CTA.
// Draws are therefore spread over all CTAs dynamically, overlap the tail of the statistics pass,
// and find their rows in L2 whenever the batch fits there.  CTAs only ever wait for records of
// rows whose units belong to CTAs of the same launch (grid <= SM count, one CTA per SM).
constexpr int DQ = 8;                           // draw descriptors in flight inside a CTA
constexpr int QD = 2;                           // slab-sum buffers between workers and the draw epilogue
constexpr uint32_t RECORD_POLLS = 1u << 22;     // bound on the wait for a queue record

struct DrawDesc {
    int kind;                                   // 0 end of stream, 1 residual draw, 2 draw from the target row
    int b, n;
    float u01;
    Norm np, nq;
};
struct FusedShared {
    StreamShared st;
    unsigned long long dslot_full[QD];
    unsigned long long dslot_empty[QD];
    DrawDesc desc[DQ];
};

// The record of row b (called by one lane): a single word {epoch, mode, n}, so that publishing it
// is one release store and reading it needs no second access.
__device__ __forceinline__ int record_stamp(uint32_t epoch, int mode, int n) {
    return (int)(((epoch & 0xffffffu) << 8) | ((uint32_t)mode << 6) | (uint32_t)n);
}
__device__ __forceinline__ void push_record(const VerifyParams& P, int b, int n, int mode) {
    st_release(&P.task_ready[b], record_stamp(P.epoch, mode, mode ? n : 0));
}

// next_unit for the fused kernel's reporting warp: a row with a bad length also gets its record.
__device__ __forceinline__ bool next_unit_fused(const VerifyParams& P, const int* cand_L, int& k, int ncand, Unit& out,
                                                bool report) {
    for (; k < ncand; ++k) {
        const int u = blockIdx.x + k * gridDim.x;
        const int i = u / P.B, b = u - i * P.B;
        const int L = k < MAX_CAND ? cand_L[k] : (P.lens ? P.lens[b] : P.K);
        if (L < 0 || L > P.K) {
            if (report && i == 0) {
                atomicOr(P.status, SPECDEC_DATA_BAD_LENGTH);
                P.n_acc[b] = -1;
                P.next[b] = -1;
                if (P.rmass) P.rmass[b] = 0.f;
                push_record(P, b, 0, 0);
            }
            continue;
        }
        if (i > L) continue;
        out.b = b; out.i = i; out.L = L; out.bonus = (i == L);
        return true;
    }
    return false;
}

template <typename T>
__global__ void __launch_bounds__(STREAM_THREADS, 1) verify_fused_kernel(const VerifyParams P) {
    constexpr int N = Elem<T>::EPV;
    extern __shared__ __align__(1024) unsigned char smem[];
    FusedShared& fs = *reinterpret_cast<FusedShared*>(smem + RING_BYTES);
    StreamShared& ss = fs.st;
    const int nvec_row = (P.V + N - 1) / N;
    const int nslab = (nvec_row + 31) / 32;
    float* slab_base = reinterpret_cast<float*>(smem + RING_BYTES + sizeof(FusedShared));   // [QD][nslab]
    const uint32_t ring = smem_u32(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    stream_init(ss, tid);
    if (tid == 0) {
        for (int s = 0; s < QD; ++s) {
            mbar_init(smem_u32(&fs.dslot_full[s]), NS);
            mbar_init(smem_u32(&fs.dslot_empty[s]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int total = (P.K + 1) * P.B;
    const int ncand = (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    for (int k = tid; k < min(ncand, MAX_CAND); k += STREAM_THREADS) {
        const int u = blockIdx.x + k * gridDim.x;
        ss.cand_L[k] = P.lens ? P.lens[u % P.B] : P.K;
    }
    __syncthreads();

    const uint32_t row_bytes = (uint32_t)P.V * sizeof(T);
    const int ntiles = (row_bytes + TILE_BYTES - 1) / TILE_BYTES;
    int k = 0;
    Unit un;

    if (warp == NS) {
        // ================================================================== producer
        if (lane != 0) return;
        const unsigned char* tbase = static_cast<const unsigned char*>(P.target);
        const unsigned char* dbase = static_cast<const unsigned char*>(P.draft);
        uint32_t stage = 0, phase = 0;
        while (next_unit(P, ss.cand_L, k, ncand, un, false)) {
            produce_unit(ss, ring, tbase + ((size_t)un.b * (P.K + 1) + un.i) * row_bytes,
                         dbase + ((size_t)un.b * P.K + un.i) * row_bytes, un.bonus, row_bytes, ntiles, stage, phase,
                         P.status);
            ++k;
        }
        // ---- phase 2: draws from the global queue
        uint32_t seq2 = 0;
        for (;;) {
            const int b = atomicAdd(&P.task_ctl[3], 1);          // rows are claimed in order
            if (b >= P.B) break;
            uint32_t stamp = 0;
            bool ok = false;
            for (uint32_t it = 0; it < RECORD_POLLS; ++it) {
                stamp = (uint32_t)ld_acquire(&P.task_ready[b]);
                if ((ok = ((stamp >> 8) == (P.epoch & 0xffffffu)))) break;
                __nanosleep(200);
            }
            if (!ok) { atomicOr(P.status, SPECDEC_DATA_WAIT_LIMIT); continue; }
            const int mode = (int)((stamp >> 6) & 3u), n = (int)(stamp & 63u);
            if (mode == 0) continue;
            const float4 r1 = __ldcg(&P.norms[(size_t)b * (P.K + 1) + n]);
            const float u01 = __ldcg(&P.uniforms[(size_t)b * (P.K + 1) + P.K]);
            // the descriptor must be in place before the unit's first tile can complete
            mbar_wait(smem_u32(&ss.empty[stage]), phase ^ 1u, P.status);
            DrawDesc& d = fs.desc[seq2 % DQ];
            d.kind = mode; d.b = b; d.n = n; d.u01 = u01;
            d.np = Norm{r1.x, r1.y}; d.nq = Norm{r1.z, r1.w};
            produce_unit(ss, ring, tbase + ((size_t)b * (P.K + 1) + n) * row_bytes,
                         dbase + ((size_t)b * P.K + n) * row_bytes, mode == 2, row_bytes, ntiles, stage, phase, P.status);
            ++seq2;
        }
        // end marker: an empty stage whose descriptor says "stop"
        mbar_wait(smem_u32(&ss.empty[stage]), phase ^ 1u, P.status);
        fs.desc[seq2 % DQ].kind = 0;
        mbar_arrive(smem_u32(&ss.full[stage]));
        // the last producer to finish empties the queue counters for the next call
        __threadfence();
        if (atomicAdd(&P.task_ctl[4], 1) == (int)gridDim.x - 1) {
            P.task_ctl[3] = 0;
            P.task_ctl[4] = 0;
        }
        return;
    }

    if (warp < NS) {
        // ================================================================== worker warps
        uint32_t stage = 0, phase = 0;
        stats_workers<T>(P, ss, ring, row_bytes, ntiles, ncand, tid, lane, warp, stage, phase);
        // ---- phase 2: draw units, described by the producer's descriptors
        for (uint32_t seq2 = 0;; ++seq2) {
            mbar_wait_warp(smem_u32(&ss.full[stage]), phase, P.status, lane);     // first tile (or the end marker)
            const DrawDesc d = fs.desc[seq2 % DQ];
            const uint32_t slot = seq2 % QD, use = seq2 / QD;
            if (use > 0) mbar_wait_warp(smem_u32(&fs.dslot_empty[slot]), (use - 1) & 1u, P.status, lane);
            if (d.kind == 0) {                     // pass the end marker on to the draw epilogue
                if (lane == 0) mbar_arrive(smem_u32(&fs.dslot_full[slot]));
                break;
            }
            float* slab_sum = slab_base + (size_t)slot * nslab;
            for (int tl = 0; tl < ntiles; ++tl) {
                const uint32_t bytes = min((uint32_t)TILE_BYTES, row_bytes - (uint32_t)tl * TILE_BYTES);
                const int nvec = bytes >> 4;
                const uint32_t base = ring + stage * (2 * TILE_BYTES);
                if (tl > 0) mbar_wait_warp(smem_u32(&ss.full[stage]), phase, P.status, lane);
#pragma unroll
                for (int j = 0; j < ITERS; ++j) {
                    const int v = tid + j * NST;         // warp-aligned: one slab per warp and j
                    float ls = 0.f;
                    if (v < nvec) {
                        float xt[N], xd[N], w[N];
                        unpack(lds128(base + v * 16), xt);
                        if (d.kind == 1) unpack(lds128(base + TILE_BYTES + v * 16), xd);
                        else {
#pragma unroll
                            for (int q = 0; q < N; ++q) xd[q] = 0.f;
                        }
                        ls = vec_weights<N>(xt, xd, P.c, d.np, d.nq, d.kind, w);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, o);
                    const int slab = tl * (TILE_BYTES / 16 / 32) + j * NS + warp;
                    if (lane == 0 && slab < nslab) slab_sum[slab] = ls;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ss.empty[stage]));
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (lane == 0) mbar_arrive(smem_u32(&fs.dslot_full[slot]));
        }
        return;
    }

    // ====================================================================== epilogue warps
    const int e = warp - NS - 1;
    uint32_t walked = 0;
    bool have = next_unit_fused(P, ss.cand_L, k, ncand, un, e == 0 && lane == 0);
    for (;;) {
        uint32_t seq = 0;
        if (lane == 0) seq = atomicAdd(&ss.next_seq, 1u);
        seq = __shfl_sync(0xffffffffu, seq, 0);
        while (have && walked < seq) {
            ++k;
            have = next_unit_fused(P, ss.cand_L, k, ncand, un, e == 0 && lane == 0);
            ++walked;
        }
        if (!have) break;
        const T* trow = static_cast<const T*>(P.target) + ((size_t)un.b * (P.K + 1) + un.i) * (size_t)P.V;
        const T* drow = un.bonus ? trow : static_cast<const T*>(P.draft) + ((size_t)un.b * P.K + un.i) * (size_t)P.V;
        int y_ok = 1;
        float t_y = 0.f, d_y = 0.f, r = 0.f;
        if (lane == 0 && !un.bonus) {
            r = P.uniforms[(size_t)un.b * (P.K + 1) + un.i];
            const int y = P.tokens[(size_t)un.b * P.K + un.i];
            y_ok = (y >= 0 && y < P.V);
            if (y_ok) { t_y = to_float(trow[y]); d_y = to_float(drow[y]); }
        }
        const uint32_t slot = seq % QSLOTS, use = seq / QSLOTS;
        mbar_wait_relaxed(smem_u32(&ss.slot_full[slot]), use & 1u, P.status, lane);
        Acc a = acc_init(), b = acc_init();
        if (lane < NS) {
            const float4 v = ss.slots[slot][lane];
            a = Acc{v.x, v.y};
            b = Acc{v.z, v.w};
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ss.slot_empty[slot]));
        a = warp_merge(a);
        b = warp_merge(b);
        if (lane == 0) {
            const Norm np = make_norm(a), nq = un.bonus ? np : make_norm(b);
            P.norms[(size_t)un.b * (P.K + 1) + un.i] = make_float4(np.rs, np.inv, nq.rs, nq.inv);
        }
        unit_accept(P, un, a, b, t_y, d_y, y_ok, r, lane);
        if (!row_arrive(P, un, lane)) continue;
        int n, bad;
        row_resolve(P, un, lane, n, bad);
        if (lane == 0) {
            P.n_acc[un.b] = bad ? -1 : n;
            if (bad) {
                P.next[un.b] = -1;
                if (P.rmass) P.rmass[un.b] = 0.f;
            }
            push_record(P, un.b, n, bad ? 0 : (n < un.L ? 1 : 2));
        }
    }
    if (e != 0) return;
    // ---- phase 2: one epilogue warp picks the tokens of the CTA's draw units
    for (uint32_t seq2 = 0;; ++seq2) {
        const uint32_t slot = seq2 % QD, use = seq2 / QD;
        mbar_wait_relaxed(smem_u32(&fs.dslot_full[slot]), use & 1u, P.status, lane);
        const DrawDesc d = fs.desc[seq2 % DQ];
        if (d.kind == 0) break;
        const int L = P.lens ? P.lens[d.b] : P.K;
        float* slab_sum = slab_base + (size_t)slot * nslab;
        const T* trow = static_cast<const T*>(P.target) + ((size_t)d.b * (P.K + 1) + d.n) * (size_t)P.V;
        const T* drow = d.kind == 2 ? trow : static_cast<const T*>(P.draft) + ((size_t)d.b * P.K + d.n) * (size_t)P.V;
        double total;
        int tok = draw_select<T, true>(P, trow, drow, d.kind, d.u01, d.np, d.nq, slab_sum, lane, &total);
        const double mass = total;
        if (d.kind == 1 && !(total > 1e-30)) {        // p == q to rounding: draw from p itself (rare)
            __shared__ UnitShared fallback_sh;
            if (lane == 0) { fallback_sh.np = d.np; fallback_sh.nq = d.nq; }
            __syncwarp();
            unit_draw<T, true>(P, trow, drow, 2, d.u01, fallback_sh, slab_sum, lane, 32, 2);
            tok = fallback_sh.token;
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(smem_u32(&fs.dslot_empty[slot]));
            P.next[d.b] = tok;
            if (P.rmass) P.rmass[d.b] = d.n >= L ? 1.f : (float)mass;
        }
    }
}

size_t fused_smem(int V, int elem_size) {
    const int epv = 16 / elem_size;
    const int nslab = ((V + epv - 1) / epv + 31) / 32;
    return (size_t)RING_BYTES + sizeof(FusedShared) + (size_t)QD * nslab * sizeof(float);
}

template <typename T>
cudaError_t launch_fused_t(const VerifyParams& p, int sm_count, size_t smem, cudaStream_t s) {
    cudaError_t e = cudaFuncSetAttribute(verify_fused_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int total = (p.K + 1) * p.B;
    verify_fused_kernel<T><<<total < sm_count ? total : sm_count, STREAM_THREADS, smem, s>>>(p);
    return cudaGetLastError();
}

// Self-test of the bounded waits: one thread waits on an mbarrier that nothing will ever complete,
// with a small poll budget, and must come back with SPECDEC_DATA_WAIT_LIMIT set.
__global__ void wait_limit_selftest_kernel(uint32_t* status, uint32_t polls) {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        bool ok = false;
        for (uint32_t it = 0; it < polls && !(ok = mbar_try_wait(smem_u32(&bar), 0)); ++it) {}
        if (!ok) atomicOr(status, SPECDEC_DATA_WAIT_LIMIT);
    }
}

size_t stream_smem(int V, int elem_size) {
    const int epv = 16 / elem_size;
    const int nslab = ((V + epv - 1) / epv + 31) / 32;
    return (size_t)RING_BYTES + sizeof(StreamShared) + (size_t)2 * nslab * sizeof(float);
}

template <typename T>
cudaError_t launch_t(const VerifyParams& p, int sm_count, size_t smem, cudaStream_t s) {
    cudaError_t e = cudaFuncSetAttribute(verify_stream_stats_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(verify_stream_draw_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int total = (p.K + 1) * p.B;
    verify_stream_stats_kernel<T><<<total < sm_count ? total : sm_count, STREAM_THREADS, smem, s>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    verify_stream_draw_kernel<T><<<p.B < sm_count ? p.B : sm_count, STREAM_THREADS, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

bool verify_stream_supported(const VerifyParams& p, specdec_dtype dtype) {
    const int es = dtype == SPECDEC_BF16 ? 2 : 4;
    if (((size_t)p.V * es) % 16 != 0) return false;
    if (reinterpret_cast<uintptr_t>(p.target) % 16 != 0 || reinterpret_cast<uintptr_t>(p.draft) % 16 != 0) return false;
    return stream_smem(p.V, es) <= 227 * 1024 && fused_smem(p.V, es) <= 227 * 1024;
}

cudaError_t launch_verify_fused(const VerifyParams& p, specdec_dtype dtype, int sm_count, cudaStream_t s,
                                int* n_launch) {
    *n_launch = 1;
    const int es = dtype == SPECDEC_BF16 ? 2 : 4;
    const size_t smem = fused_smem(p.V, es);
    return dtype == SPECDEC_BF16 ? launch_fused_t<__nv_bfloat16>(p, sm_count, smem, s) : launch_fused_t<float>(p, sm_count, smem, s);
}

cudaError_t launch_verify_stream(const VerifyParams& p, specdec_dtype dtype, int sm_count, cudaStream_t s,
                                 int* n_launch) {
    *n_launch = 2;
    const int es = dtype == SPECDEC_BF16 ? 2 : 4;
    const size_t smem = stream_smem(p.V, es);
    return dtype == SPECDEC_BF16 ? launch_t<__nv_bfloat16>(p, sm_count, smem, s) : launch_t<float>(p, sm_count, smem, s);
}

cudaError_t launch_wait_limit_selftest(uint32_t* status, cudaStream_t s) {
    wait_limit_selftest_kernel<<<1, 32, 0, s>>>(status, 4096u);
    return cudaGetLastError();
}
