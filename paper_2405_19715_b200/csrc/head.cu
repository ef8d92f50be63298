// Acceptance-prediction head (Eq. 3 and Section 5.1 of arXiv 2405.19715):
//   x_k = x_{k-1} + SiLU(W_k x_{k-1} + b_k), k = 1..D;  accept_prob = sigmoid(w_out . x_D + b_out).
//
// Each residual block is one GEMM  Z[M, d] = X[M, d] * W^T  (W stored [out, in], so both operands
// are K-major) on the 5th-generation tensor cores: operand tiles arrive in shared memory by TMA
// (128-byte swizzle), one thread issues tcgen05.mma with the fp32 accumulator in tensor memory,
// and eight epilogue warps read the (double-buffered) accumulator back with tcgen05.ld and apply
// bias, SiLU and the residual while the next tile's MMAs run.  The last block does not store x_D: its
// epilogue multiplies by w_out and leaves one partial dot product per (row, column tile); whoever
// finishes a row's last tile adds them and applies the sigmoid.  D = 0 is a plain row-times-vector kernel.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "specdec_internal.h"

namespace {

constexpr int BM = 128;                  // rows of X per CTA (= UMMA M)
constexpr int BK = 64;                   // bf16 elements per k-block: one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int EPI_WARPS = 8;             // two per 32-lane quarter of tensor memory, each taking half the columns
constexpr int HEAD_THREADS = (2 + EPI_WARPS) * 32;   // warp 0 TMA, warp 1 MMA + tensor-memory owner, then epilogue
constexpr uint32_t WAIT_POLLS = 1u << 24;
constexpr int OUT_COLS = 32, OUT_ROWS = 32;                       // box of one TMA store of the output: 32 rows x 64 bytes
constexpr int OUT_BOX_BYTES = OUT_ROWS * OUT_COLS * 2;

// PAIR: two CTAs (a cluster) share a 256 x BN tile; each loads its 128 rows of X and its half of the tile's
// weight rows, and one thread of the even CTA issues M = 256 MMAs over both CTAs' shared and tensor memory.
template <int BN, bool PAIR> struct Cfg {
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = (PAIR ? BN / 2 : BN) * BK * 2;
    static constexpr int KB_BYTES = A_BYTES + B_BYTES;                // operands of one k-block
    // k-blocks per ring stage, i.e. per barrier round trip of the issuing thread: with the pair's smaller operands
    // two k-blocks (eight MMAs) share one wait and one commit and the ring still holds three stages
    static constexpr int KSUB = PAIR ? 2 : 1;
    static constexpr int STAGE_BYTES = KSUB * KB_BYTES;
    static constexpr int STAGES = 192 * 1024 / STAGE_BYTES;           // 4 x 48 KB or 6 x 32 KB; pairs: 3 x 64 KB or 4 x 48 KB
    static constexpr int OUT_BYTES = EPI_WARPS * 2 * OUT_BOX_BYTES;   // two output boxes per epilogue warp
    static constexpr int SMEM = STAGES * STAGE_BYTES + OUT_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
};

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
// Bounded wait: when the polls run out the thread simply continues, so it still reaches the barriers and
// the tensor-memory release below; `budget` is the calling thread's poll allowance, cut to WAIT_POLLS_LEFT by
// a give-up, so that a broken pipeline drains in about a second instead of one limit per wait, and
// report_wait_limit() at the end of the kernel turns a cut allowance into the status bit.
// The wait is only a probe loop on registers: in the MMA-issuing thread the barrier has nearly always
// completed already, and with the status update inside the wait that thread needed ~100 cycles more per
// k-block than the tensor pipe does (measured: 643 against 547 cycles per k-block, 512 being the pipe's).
constexpr uint32_t WAIT_POLLS_LEFT = 1024;
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, uint32_t& budget) {
    for (uint32_t n = 0; !mbar_try_wait(bar, parity); ++n)
        if (n >= budget) {
            budget = WAIT_POLLS_LEFT;
            return;
        }
}
__device__ __forceinline__ void report_wait_limit(uint32_t* status, uint32_t budget) {
    if (budget != WAIT_POLLS) atomicOr(status, SPECDEC_DATA_WAIT_LIMIT);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled: start
// address >> 4 in bits 0-13, leading offset 16 B (unused by swizzled layouts) in bit 16; in the high word
// 1024 B between 8-row groups, descriptor version 1, layout type SWIZZLE_128B.
// The four MMAs of one 64-wide k-block in one statement.  `a_lo`, `b_lo` are the low words of the operands'
// descriptors at k = 0; a step of 16 bf16 along K is 32 bytes, i.e. + 2 in that word, and the high word is
// the same for every tile, so the issuing thread spends one add per descriptor instead of rebuilding 64-bit
// values.  `acc_first` is the
// accumulate flag of the first MMA (0 on a tile's first k-block); the other three always accumulate.
constexpr uint32_t UMMA_DESC_HI = 64u | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr) { return ((smem_addr >> 4) & 0x3FFFu) | (1u << 16); }
__device__ __forceinline__ void umma_kblock(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.eq.b32 q, 0, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, q;\n\t"
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, q;\n\t"
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, q;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(acc_first), "r"(UMMA_DESC_HI) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- the same for a pair of CTAs (cta_group::2) ----
__device__ __forceinline__ uint32_t pair_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void pair_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The address of this CTA's shared-memory location `a` in CTA `rank` of the pair.
__device__ __forceinline__ uint32_t pair_map(uint32_t a, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
    return r;
}
// TMA load by one CTA of a pair whose bytes are counted on the EVEN CTA's barrier (peer bit of the barrier's
// cluster address cleared).  Each CTA fetches its own operands.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar & 0xFEFFFFFFu) : "memory");
}
__device__ __forceinline__ void umma_kblock_pair(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t.reg .b32 ta, tb;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.eq.b32 q, 0, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, p;\n\t"
        "add.u32 ta, %1, 2;\n\tadd.u32 tb, %2, 2;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t"
        "add.u32 ta, %1, 4;\n\tadd.u32 tb, %2, 4;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t"
        "add.u32 ta, %1, 6;\n\tadd.u32 tb, %2, 6;\n\t"
        "mov.b64 da, {ta, %5};\n\tmov.b64 db, {tb, %5};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(acc_first), "r"(UMMA_DESC_HI) : "memory");
}
// Arrive on the barrier at this offset in both CTAs of the pair once the pair's MMAs issued so far have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__host__ __device__ constexpr uint32_t umma_idesc_pair(int n) {           // M = 256 across the pair
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float silu(float z) { return __fdividef(z, 1.f + __expf(-z)); }
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

struct BlockParams {
    const __nv_bfloat16* X;      // [M, d] input of the block (also the residual)
    const __nv_bfloat16* bias;   // [d] or null
    __nv_bfloat16* Y;            // [M, d] output, null for the last block
    const __nv_bfloat16* w_out;  // [d], last block only
    float* partial;              // [M, 2 * d / BN], last block only
    int M, d;
    uint32_t* status;
    // weights-as-M kernel, last block: the CTA that finishes last adds the partial dots and applies the sigmoid
    int32_t* done_ctr;
    float* accept_prob;
    float b_out;
};

// Per-tile timestamps of the first and the last CTA (diagnostic builds only): [CTA 0 / last][tile][slot], ns of
// the global timer.  Slots: 0 TMA warp requests the tile's first k-block, 1 MMA warp has a free accumulator,
// 2 first k-block landed, 3 all MMAs issued, 4 epilogue sees the accumulator complete, 5 epilogue done;
// 6 and 7 hold the SM's cycle counter at stamps 2 and 3 (cycles of the main loop, and with the timer its clock).
#ifdef SPECDEC_STAMPS
__device__ long long head_tile_stamps[2 * 8 * 8];
#define TILE_STAMP(it, slot)                                                                          \
    do {                                                                                              \
        if ((blockIdx.x == 0 || blockIdx.x == gridDim.x - 1) && (it) < 8) {                           \
            long long t_;                                                                             \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                    \
            head_tile_stamps[((blockIdx.x == 0 ? 0 : 1) * 8 + (it)) * 8 + (slot)] = t_;               \
            if ((slot) == 2 || (slot) == 3)                                                           \
                head_tile_stamps[((blockIdx.x == 0 ? 0 : 1) * 8 + (it)) * 8 + (slot) + 4] = clock64(); \
        }                                                                                             \
    } while (0)
#else
#define TILE_STAMP(it, slot) do {} while (0)
#endif

// The residual blocks of one call as ONE launch (more than 256 rows).
constexpr int CHAIN_MAX = 8;                       // residual blocks per launch (the entry point's depth limit)
constexpr uint32_t FLAG_POLLS = 1u << 21;          // polls of a row block's counter before giving up (~ a second)
struct ChainLayer {
    const __nv_bfloat16* X;      // [M, d] input of the block (also the residual)
    const __nv_bfloat16* bias;   // [d] or null
    __nv_bfloat16* Y;            // [M, d] output; null for the block that ends the head
};
struct ChainParams {
    CUtensorMap mapX[CHAIN_MAX], mapW[CHAIN_MAX];
    CUtensorMap mapY[CHAIN_MAX];     // output of a block as 32 x 32 boxes, 64-byte swizzle (unused for the head's last block)
    ChainLayer layer[CHAIN_MAX];
    int first, end;              // blocks [first, end) are computed by this launch
    int depth;                   // blocks of the head: block depth - 1 multiplies by w_out instead of storing
    int M, d;
    const __nv_bfloat16* w_out;  // [d]
    float* partial;              // [M, 2 * d / BN] partial dots of the last block
    uint32_t* ready;             // [depth][row blocks] epilogue warps that have finished a tile of (block, row block); zero at
                                 // launch, and cleared again by the CTA that leaves last (so a launch may be replayed from a graph)
    uint32_t* exited;            // CTAs of this launch that have left
    float* accept_prob;
    float b_out;
    uint32_t* status;
};

__device__ __forceinline__ uint4 ld_residual(const uint4* p, bool past_l1) { return past_l1 ? __ldcg(p) : *p; }
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Persistent over the tiles of all its blocks: tile g = (block, row block, column tile), column tile fastest,
// block slowest; worker w (a CTA, or with PAIR a cluster of two CTAs that share a 256-row tile, each loading
// and finishing its own 128 rows) works on tiles w, w + workers, ...  A CTA's part of a tile of block l > first
// reads 128 rows that the tiles of block l - 1 in the same row block wrote, so its TMA thread first waits until
// `ready` shows all of them finished (every epilogue warp counts once per tile, after its stores).  Those tiles
// come earlier in the order, so with all CTAs resident (the launch is cooperative) the tile with the lowest
// unfinished index never waits for an unfinished one; the wait is bounded all the same.  With 512 tiles per
// block on 148 SMs two blocks take 7 rounds in one launch instead of 4 + 4 in two, and only the first tile of
// the launch waits for its operands with nothing to overlap.  The accumulator is double-buffered in tensor memory (2 x BN columns), so
// the epilogue of one tile runs while the MMAs of the next are issued.  In the head's last block the warp that
// completes a row block's count adds the block's partial dots in column order and applies the sigmoid.
template <int BN, bool PAIR>
__global__ void __launch_bounds__(HEAD_THREADS, 1)
head_chain_kernel(const __grid_constant__ ChainParams P) {
    using C = Cfg<BN, PAIR>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
    unsigned char* aligned = smem_raw + (base - smem_u32(smem_raw));
    unsigned char* out_stage = aligned + C::STAGES * C::STAGE_BYTES;      // [epilogue warp][2][32 rows][64 bytes]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(out_stage + C::OUT_BYTES);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * C::STAGES, tfull0 = empty0 + 8 * C::STAGES,
                   tempty0 = tfull0 + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int TM = PAIR ? 2 * BM : BM;                                // rows of a tile
    const uint32_t rank = PAIR ? pair_rank() : 0u;                        // 0: issues the pair's MMAs, owns its barriers
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;   // a CTA or a pair of CTAs
    const int nworkers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int nkb = P.d / BK;
    const int ntn = P.d / BN, ntm = (P.M + TM - 1) / TM, per_block = ntn * ntm;
    const int nrb = ntm * (TM / BM);                                      // 128-row blocks with a counter (the last may be empty)
    const int ntiles = (P.end - P.first) * per_block;
    const uint32_t tile_warps = (uint32_t)(ntn * EPI_WARPS);              // counts that complete a row block
    uint32_t budget = WAIT_POLLS;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull0 + 8 * b, 1);
            mbar_init(tempty0 + 8 * b, PAIR ? 2 * EPI_WARPS : EPI_WARPS);   // a pair: the even CTA's, for both epilogues
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                      // this warp owns the tensor-memory allocation (of a pair: the same warp of both CTAs)
        if constexpr (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)(2 * BN)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)(2 * BN)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) pair_sync();      // both CTAs' barriers exist before anything is sent to them
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, it = 0;
            bool wrapped = false;                              // the ring has been gone round at least once
            for (int g = worker; g < ntiles; g += nworkers, ++it) {
                const int l = P.first + g / per_block, t = g % per_block;
                const int m0 = (t / ntn) * TM + (int)rank * BM;                         // this CTA's rows of X
                const int n0 = (t % ntn) * BN + (PAIR ? (int)rank * (BN / 2) : 0);      // ... and rows of W
                if (l > P.first) {                             // the rows of X come from this launch's previous block
                    const uint32_t* ctr = P.ready + (size_t)(l - 1) * nrb + m0 / BM;
                    uint32_t polls = 0;
                    while (ld_acquire_u32(ctr) < tile_warps)
                        if (++polls >= (budget == WAIT_POLLS ? FLAG_POLLS : WAIT_POLLS_LEFT)) {
                            budget = WAIT_POLLS_LEFT;
                            break;
                        }
                    asm volatile("fence.proxy.async;" ::: "memory");   // the loads below go through the async proxy
                }
                const CUtensorMap* mx = &P.mapX[l];
                const CUtensorMap* mw = &P.mapW[l];
                for (int ks = 0; ks < nkb / C::KSUB; ++ks) {
                    mbar_wait(empty0 + 8 * stage, phase ^ 1u, budget);
                    if (ks == 0) TILE_STAMP(it, 0);
                    if constexpr (PAIR) {                      // both CTAs' bytes complete the even CTA's barrier
                        if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * C::STAGE_BYTES);
                    } else {
                        mbar_expect_tx(full0 + 8 * stage, C::STAGE_BYTES);
                    }
#pragma unroll
                    for (int h = 0; h < C::KSUB; ++h) {
                        const uint32_t a = base + stage * C::STAGE_BYTES + h * C::KB_BYTES, b = a + C::A_BYTES;
                        const int k0 = (ks * C::KSUB + h) * BK;
                        if constexpr (PAIR) {
                            tma_load_2d_pair(a, mx, k0, m0, full0 + 8 * stage);
                            tma_load_2d_pair(b, mw, k0, n0, full0 + 8 * stage);
                        } else {
                            tma_load_2d(a, mx, k0, m0, full0 + 8 * stage);
                            tma_load_2d(b, mw, k0, n0, full0 + 8 * stage);
                        }
                    }
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1u; wrapped = true; }
                }
            }
            // Before this CTA may end, every copy it asked for has landed and been consumed: each stage's last
            // load (on the CTA that owns the full barrier) and the MMAs that read it.  All of it has happened
            // long ago unless a wait gave up, in which case these waits are short as well.
            for (uint32_t s = 0; s < (uint32_t)C::STAGES; ++s) {
                if (s >= stage && !wrapped) continue;           // never used
                const uint32_t ph = s < stage ? phase : phase ^ 1u;
                if (rank == 0) mbar_wait(full0 + 8 * s, ph, budget);
                mbar_wait(empty0 + 8 * s, ph, budget);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = PAIR ? umma_idesc_pair(BN) : umma_idesc(BN);
            static_assert(BK / UMMA_K == 4, "umma_kblock issues four MMAs");
            const uint32_t desc_lo0 = umma_desc_lo(base);      // stage 0 of the ring, operand A, k = 0
            uint32_t stage = 0, phase = 0, it = 0;
            for (int g = worker; g < ntiles; g += nworkers, ++it) {
                const uint32_t buf = it & 1u, use = (it >> 1) & 1u;
                mbar_wait(tempty0 + 8 * buf, use ^ 1u, budget);      // epilogue has drained this accumulator
                TILE_STAMP(it, 1);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem + buf * BN;
                for (int ks = 0; ks < nkb / C::KSUB; ++ks) {
                    mbar_wait(full0 + 8 * stage, phase, budget);
                    if (ks == 0) TILE_STAMP(it, 2);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                    for (int h = 0; h < C::KSUB; ++h) {
                        const uint32_t a_lo = desc_lo0 + stage * (C::STAGE_BYTES >> 4) + h * (C::KB_BYTES >> 4);
                        if constexpr (PAIR) umma_kblock_pair(acc, a_lo, a_lo + (C::A_BYTES >> 4), idesc, (ks | h) != 0 ? 1u : 0u);
                        else umma_kblock(acc, a_lo, a_lo + (C::A_BYTES >> 4), idesc, (ks | h) != 0 ? 1u : 0u);
                    }
                    if constexpr (PAIR) umma_commit_pair(empty0 + 8 * stage);   // stage reusable, in both CTAs, once these MMAs have read it
                    else umma_commit(empty0 + 8 * stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
                }
                if constexpr (PAIR) umma_commit_pair(tfull0 + 8 * buf);   // accumulator complete (in both CTAs)
                else umma_commit(tfull0 + 8 * buf);
                TILE_STAMP(it, 3);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int q = warp & 3;                            // tensor-memory lane quarter this warp may read
        const int half = (warp - 2) >> 2;                  // which half of the tile's columns
        constexpr int CH = BN / 32 / 2;                    // 32-column chunks per warp
        uint32_t it = 0;
        for (int g = worker; g < ntiles; g += nworkers, ++it) {
            const int l = P.first + g / per_block, t = g % per_block;
            const int m0 = (t / ntn) * TM + (int)rank * BM, n0 = (t % ntn) * BN;
            const bool last = l == P.depth - 1;
            const __nv_bfloat16* bias = P.layer[l].bias;
            const __nv_bfloat16* w_out = last ? P.w_out : nullptr;
            __nv_bfloat16* Y = P.layer[l].Y;
            const uint32_t buf = it & 1u, use = (it >> 1) & 1u;
            const int m = m0 + q * 32 + lane;
            const bool row_ok = m < P.M;
            // The residual was written by other SMs during this launch if l > first.  This SM's L1 can only hold
            // an older version of those rows if it read the same buffer before it was rewritten, i.e. from the
            // fourth block of a launch on (two buffers alternate): those reads go past L1.
            const bool past_l1 = l >= P.first + 3;
            const uint4* xrow = reinterpret_cast<const uint4*>(P.layer[l].X + (size_t)(row_ok ? m : 0) * P.d + n0);
            uint4 xv[4], xn[4];
            mbar_wait(tfull0 + 8 * buf, use, budget);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (warp == 2 && lane == 0) TILE_STAMP(it, 4);
#pragma unroll
            for (int j = 0; j < 4; ++j) xn[j] = row_ok ? ld_residual(xrow + (half * CH) * 4 + j, past_l1) : make_uint4(0, 0, 0, 0);
            float dot = 0.f;
#pragma unroll 1
            for (int cc = 0; cc < CH; ++cc) {
                const int c = half * CH + cc;
                float acc[32];
                tmem_ld32(tmem + buf * BN + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), acc);
                uint4 bv[4], wv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    xv[j] = xn[j];
                    if (cc + 1 < CH) xn[j] = row_ok ? ld_residual(xrow + (c + 1) * 4 + j, past_l1) : make_uint4(0, 0, 0, 0);
                    bv[j] = bias ? __ldg(reinterpret_cast<const uint4*>(bias + n0 + c * 32) + j) : make_uint4(0, 0, 0, 0);
                    wv[j] = w_out ? __ldg(reinterpret_cast<const uint4*>(w_out + n0 + c * 32) + j) : make_uint4(0, 0, 0, 0);
                }
                const uint32_t* xw = reinterpret_cast<const uint32_t*>(xv);
                const uint32_t* bw = reinterpret_cast<const uint32_t*>(bv);
                const uint32_t* ww = reinterpret_cast<const uint32_t*>(wv);
                uint32_t out[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float y0 = bf16lo(xw[j]) + silu(acc[2 * j] + bf16lo(bw[j]));
                    const float y1 = bf16hi(xw[j]) + silu(acc[2 * j + 1] + bf16hi(bw[j]));
                    dot = fmaf(y0, bf16lo(ww[j]), dot);
                    dot = fmaf(y1, bf16hi(ww[j]), dot);
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(y0, y1);
                    out[j] = *reinterpret_cast<const uint32_t*>(&pk);
                }
                if (Y && m0 + q * 32 < P.M) {                  // warp-uniform; rows past M are clipped by the store
                    // The warp's 32 rows x 64 bytes go to shared memory (64-byte swizzle: 16-byte chunk j of row r
                    // at chunk j ^ ((r >> 1) & 3), conflict-free) and from there to Y as one TMA store; two boxes
                    // alternate, a box being rewritten once the store before last has read it.
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                    unsigned char* box = out_stage + ((warp - 2) * 2 + (cc & 1)) * OUT_BOX_BYTES;
                    uint4* brow = reinterpret_cast<uint4*>(box + lane * (OUT_COLS * 2));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        brow[j ^ ((lane >> 1) & 3)] = make_uint4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&P.mapY[l], smem_u32(box), n0 + c * 32, m0 + q * 32);
                }
            }
            // this warp has read its part of the accumulator: hand the buffer back to the MMA issuer
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (PAIR && rank != 0) mbar_arrive_cluster(pair_map(tempty0 + 8 * buf, 0));
                else mbar_arrive(tempty0 + 8 * buf);
            }
            if (warp == 2 && lane == 0) TILE_STAMP(it, 5);
            if (last && row_ok) P.partial[(size_t)m * (2 * ntn) + 2 * (t % ntn) + half] = dot;
            // count this warp's part of the tile as written; the count of a row block is what the next block's
            // tiles (their TMA loads: the async proxy) and, in the last block, the row block's finisher wait for
            __syncwarp();
            uint32_t* ctr = P.ready + (size_t)l * nrb + m0 / BM;
            uint32_t before = 0;
            if (lane == 0) {
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this warp's boxes are written
                asm volatile("fence.proxy.async;" ::: "memory");            // ... through the async proxy
                __threadfence();                               // the warp's stores (ordered before by the barrier), then the count
                before = atomicAdd(ctr, 1u);
            }
            before = __shfl_sync(0xffffffffu, before, 0);
            if (last && before == tile_warps - 1) {            // every dot of this row block is in place
                __threadfence();
                for (int r = lane; r < BM; r += 32) {
                    const int mr = m0 + r;
                    if (mr >= P.M) break;
                    const float* pr = P.partial + (size_t)mr * (2 * ntn);
                    float sum = P.b_out;
                    for (int c = 0; c < 2 * ntn; ++c) sum += __ldcg(pr + c);
                    P.accept_prob[mr] = 1.f / (1.f + __expf(-sum));
                }
            }
        }
    }
    report_wait_limit(P.status, budget);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) pair_sync();      // nothing is in flight towards the other CTA's barriers or tensor memory any more
    if (warp == 2) {                      // the CTA that leaves last puts the counters back to zero
        uint32_t left = 0;
        if (lane == 0) {
            __threadfence();
            left = atomicAdd(P.exited, 1u);
        }
        left = __shfl_sync(0xffffffffu, left, 0);
        if (left == gridDim.x - 1) {
            __threadfence();
            for (int i = lane; i < P.depth * nrb; i += 32) P.ready[i] = 0;
            if (lane == 0) *P.exited = 0;
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if constexpr (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)(2 * BN)) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)(2 * BN)) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// The block for up to 256 rows (the online use of Eq. 3 in Algorithm 1's loop: one drafted token per call for one
// to hundreds of concurrent sequences):
// the GEMM is a stream of the weights against a handful of rows, so the WEIGHTS are the M-side operand.
// A tile is Z^T[128 output features, N rows of X] = W[128, k] * X^T[k, N]: one tcgen05.mma takes 128
// weight rows whatever the number of rows of X (N = M rounded up to 16); the accumulator holds one
// output feature per tensor-memory lane and one row of X per column.  To put the weight stream on as
// many SMs as the memory system needs, the reduction dimension is split over the KS CTAs of a
// thread-block cluster: each CTA accumulates its k-slice, then sends the lane quarters of its
// accumulator to the CTAs that own them (stores into the owners' shared memory), and after a cluster
// barrier each CTA adds the KS contributions to its 128 / KS features and runs the epilogue for them
// (bias, SiLU, residual, bf16 store, or the w_out dot of the last block, whose last CTA also adds the
// dots and applies the sigmoid).  The kernel is launched programmatically dependent on the stream's
// previous kernel -- the previous block -- and asks for its first ring-full of weight tiles before
// that kernel has completed; only the rows of X wait for it.
constexpr int SW_THREADS = 6 * 32;       // warp 0 TMA, warp 1 MMA + tensor-memory owner, warps 2-5 epilogue
constexpr int SW_UR = 8;                 // rows an epilogue warp works on together

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t local_addr, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// Phase timestamps of one CTA (diagnostic builds only): [last block ? 1 : 0][warp][slot], global timer in ns.
#ifdef SPECDEC_STAMPS
__device__ long long head_stamps[2 * 6 * 16];
#define HEAD_STAMP(slot)                                                                         \
    do {                                                                                         \
        if (blockIdx.x == 5 && lane == 0) {                                                      \
            long long t_;                                                                        \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                               \
            head_stamps[(P.partial ? 96 : 0) + warp * 16 + (slot)] = t_;                         \
        }                                                                                        \
    } while (0)
#else
#define HEAD_STAMP(slot) do {} while (0)
#endif

template <int KS>
__global__ void __launch_bounds__(SW_THREADS, 1)
head_swap_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW, const BlockParams P,
                 int Npad, int stages, int tmem_cols) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* aligned = smem_raw + (base - smem_u32(smem_raw));
    const int a_bytes = BM * BK * 2, stage_bytes = a_bytes + Npad * BK * 2;
    const int ring_bytes = max(stages * stage_bytes, 512 * Npad);         // the ring is reused to receive the partial sums
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(aligned + ring_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * stages, tfull = empty0 + 8 * stages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * stages + 2);
    float* recv = reinterpret_cast<float*>(aligned);                      // [KS][4 / KS][Npad][32]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    HEAD_STAMP(0);
    const int rank = (int)cluster_rank();
    const int n0 = (blockIdx.x / KS) * BM;                                // first output feature of the tile
    const int nkb = P.d / BK / KS, kb0 = rank * nkb;                      // this CTA's k-blocks
    constexpr int QL = 4 / KS;                                            // lane quarters a CTA finishes
    uint32_t budget = WAIT_POLLS;
    unsigned short xr[SW_UR];                                             // residual values fetched ahead (epilogue warps)

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(tfull, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    HEAD_STAMP(1);

    if (warp == 0) {
        if (lane == 0) {
            // The weights do not depend on the stream's previous kernel: the first ring-full of weight tiles
            // is requested before that kernel is known to be complete, the rows of X -- its output -- after.
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            const int ahead = min(stages, nkb);
            for (int kb = 0; kb < ahead; ++kb) {
                mbar_expect_tx(full0 + 8 * kb, stage_bytes);
                tma_load_2d(base + kb * stage_bytes, &mapW, (kb0 + kb) * BK, n0, full0 + 8 * kb);
            }
            HEAD_STAMP(2);
            asm volatile("griddepcontrol.wait;" ::: "memory");
            HEAD_STAMP(3);
            for (int kb = 0; kb < ahead; ++kb)
                tma_load_2d(base + kb * stage_bytes + a_bytes, &mapX, (kb0 + kb) * BK, 0, full0 + 8 * kb);
            uint32_t stage = 0, phase = 1;                                // the ring has been filled once
            for (int kb = ahead; kb < nkb; ++kb) {
                mbar_wait(empty0 + 8 * stage, phase ^ 1u, budget);
                const uint32_t a = base + stage * stage_bytes, b = a + a_bytes;
                mbar_expect_tx(full0 + 8 * stage, stage_bytes);
                tma_load_2d(a, &mapW, (kb0 + kb) * BK, n0, full0 + 8 * stage);     // 128 weight rows
                tma_load_2d(b, &mapX, (kb0 + kb) * BK, 0, full0 + 8 * stage);      // the rows of X (zeros past M)
                if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(Npad);
            uint32_t stage = 0, phase = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                mbar_wait(full0 + 8 * stage, phase, budget);
                if (kb == 0) HEAD_STAMP(2);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_lo = umma_desc_lo(base + stage * stage_bytes);
                umma_kblock(tmem, a_lo, a_lo + (a_bytes >> 4), idesc, kb != 0 ? 1u : 0u);
                umma_commit(empty0 + 8 * stage);
                if (++stage == (uint32_t)stages) { stage = 0; phase ^= 1u; }
            }
            umma_commit(tfull);
            HEAD_STAMP(3);
        }
    } else {
        // the residual values of this warp's first rows, requested while the weights stream
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const unsigned short* xcol = reinterpret_cast<const unsigned short*>(P.X) + n0 + rank * QL * 32 + lane;
#pragma unroll
        for (int u = 0; u < SW_UR; ++u) {
            const int m = (warp - 2) + 4 * u;
            xr[u] = m < P.M ? __ldg(xcol + (size_t)m * P.d) : (unsigned short)0;
        }
        mbar_wait(tfull, 0, budget);                            // this CTA's accumulator is complete
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        HEAD_STAMP(4);
    }
    __syncwarp();
    cluster_sync_all();          // every CTA of the cluster has consumed its ring: it may now be written from outside
    HEAD_STAMP(5);

    if (warp >= 2) {
        // lane quarter q of the accumulator goes to the CTA that finishes it
        const int q = warp & 3, dst = q / QL, ql = q - dst * QL;
        const uint32_t slot = smem_u32(recv) + (uint32_t)(((rank * QL + ql) * Npad) * 32 + lane) * 4u;
        for (int c0 = 0; c0 < Npad; c0 += 32) {
            float v[32];
            tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (c0 + j < P.M) st_cluster_f32(slot + (uint32_t)((c0 + j) * 32) * 4u, (uint32_t)dst, v[j]);
        }
    }
    HEAD_STAMP(6);
    __syncwarp();
    cluster_sync_all();          // all contributions have arrived
    HEAD_STAMP(7);
    const int ntile32 = P.d / 32;
    if (warp >= 2) {
        // Eight rows at a time, step by step across the eight: one warp per scheduler has nothing else to
        // hide a row's latencies behind.  The next eight residuals are requested first.
        const int e = warp - 2;
        for (int ql = 0; ql < QL; ++ql) {
            const int n = n0 + (rank * QL + ql) * 32 + lane;
            const float bias = P.bias ? __bfloat162float(P.bias[n]) : 0.f;
            const float wo = P.w_out ? __bfloat162float(P.w_out[n]) : 0.f;
            const unsigned short* xcol = reinterpret_cast<const unsigned short*>(P.X) + n;
            if (ql > 0) {
#pragma unroll
                for (int u = 0; u < SW_UR; ++u) {
                    const int m = e + 4 * u;
                    xr[u] = m < P.M ? __ldg(xcol + (size_t)m * P.d) : (unsigned short)0;
                }
            }
            for (int m0 = e; m0 < P.M; m0 += 4 * SW_UR) {
                unsigned short xn[SW_UR];
                float z[SW_UR], y[SW_UR];
#pragma unroll
                for (int u = 0; u < SW_UR; ++u) {
                    const int m = m0 + 4 * (SW_UR + u);
                    xn[u] = m < P.M ? __ldg(xcol + (size_t)m * P.d) : (unsigned short)0;
                }
#pragma unroll
                for (int u = 0; u < SW_UR; ++u) {
                    const int m = min(m0 + 4 * u, Npad - 1);
                    z[u] = bias;
#pragma unroll
                    for (int src = 0; src < KS; ++src) z[u] += recv[((src * QL + ql) * Npad + m) * 32 + lane];
                }
#pragma unroll
                for (int u = 0; u < SW_UR; ++u) y[u] = __uint_as_float((uint32_t)xr[u] << 16) + silu(z[u]);
                if (P.Y) {
#pragma unroll
                    for (int u = 0; u < SW_UR; ++u)
                        if (m0 + 4 * u < P.M) P.Y[(size_t)(m0 + 4 * u) * P.d + n] = __float2bfloat16_rn(y[u]);
                }
                if (P.partial) {
#pragma unroll
                    for (int u = 0; u < SW_UR; ++u) y[u] *= wo;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                        for (int u = 0; u < SW_UR; ++u) y[u] += __shfl_xor_sync(0xffffffffu, y[u], o);
#pragma unroll
                    for (int u = 0; u < SW_UR; ++u)
                        if (lane == u && m0 + 4 * u < P.M) P.partial[(size_t)(m0 + 4 * u) * ntile32 + (n >> 5)] = y[u];
                }
#pragma unroll
                for (int u = 0; u < SW_UR; ++u) xr[u] = xn[u];
            }
        }
    }
    HEAD_STAMP(8);
    if (P.partial) {
        // last block: the CTA that finishes last adds every row's partial dots (a warp per row, fixed order)
        // and applies the sigmoid
        __shared__ int last;
        __threadfence();
        __syncthreads();
        if (tid == 0) last = (atomicAdd(P.done_ctr, 1) == (int)gridDim.x - 1);
        __syncthreads();
        if (last) {
            __threadfence();
            for (int m = warp; m < P.M; m += SW_THREADS / 32) {
                float v = 0.f;
                for (int t = lane; t < ntile32; t += 32) v += __ldcg(P.partial + (size_t)m * ntile32 + t);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) P.accept_prob[m] = 1.f / (1.f + __expf(-(v + P.b_out)));
            }
            if (tid == 0) *P.done_ctr = 0;                                // ready for the next call
        }
    }
    report_wait_limit(P.status, budget);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    HEAD_STAMP(9);
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)tmem_cols) : "memory");
    }
}

// D = 0: one warp per row, accept_prob[m] = sigmoid(hidden[m, :] . w_out + b_out)
__global__ void head_linear_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ w, int M,
                                   int d, float b_out, float* __restrict__ accept_prob) {
    const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (m >= M) return;
    const uint4* xr = reinterpret_cast<const uint4*>(X + (size_t)m * d);
    const uint4* wr = reinterpret_cast<const uint4*>(w);
    float s = 0.f;
    for (int v = lane; v < d / 8; v += 32) {
        const uint4 a = __ldg(xr + v), b = __ldg(wr + v);
        const uint32_t* aw = reinterpret_cast<const uint32_t*>(&a);
        const uint32_t* bw = reinterpret_cast<const uint32_t*>(&b);
#pragma unroll
        for (int j = 0; j < 4; ++j) s = fmaf(bf16lo(aw[j]), bf16lo(bw[j]), fmaf(bf16hi(aw[j]), bf16hi(bw[j]), s));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) accept_prob[m] = 1.f / (1.f + __expf(-(s + b_out)));
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 2-D bf16 row-major [rows, cols] tensor, box {box_cols, box_rows} with rows of 128 bytes (128-byte swizzle) or
// 64 bytes (64-byte swizzle), zero fill outside.
bool make_map(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows, int box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, box_cols * 2 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The map of an operand, from the context's cache when this operand has been seen before.  The map is
// copied out: the next look-up may recycle the slot it came from.
bool cached_map(specdec_ctx* ctx, CUtensorMap* out, const void* ptr, int rows, int cols, int box_rows, int box_cols = BK) {
    static_assert(sizeof(CUtensorMap) <= sizeof(HeadMapEntry::map), "tensor map larger than its cache slot");
    for (HeadMapEntry& e : ctx->head_maps)
        if (e.ptr == ptr && e.rows == rows && e.cols == cols && e.box_rows == box_rows && e.box_cols == box_cols) {
            memcpy(out, e.map, sizeof(CUtensorMap));
            return true;
        }
    if (!make_map(out, ptr, rows, cols, box_rows, box_cols)) return false;
    HeadMapEntry& e = ctx->head_maps[ctx->head_map_next];
    ctx->head_map_next = (ctx->head_map_next + 1) % 32;
    memcpy(e.map, out, sizeof(CUtensorMap));
    e.ptr = ptr;
    e.rows = rows;
    e.cols = cols;
    e.box_rows = box_rows;
    e.box_cols = box_cols;
    return true;
}

cudaError_t launch_swap(const CUtensorMap& mx, const CUtensorMap& mw, const BlockParams& p, int Npad, cudaStream_t s) {
    const int nkb_all = p.d / BK;
    const int KS = nkb_all % 4 == 0 ? 4 : 2;                              // d is a multiple of 128: at least two k-blocks
    const int nkb = nkb_all / KS;
    const int stage_bytes = BM * BK * 2 + Npad * BK * 2;
    // Two CTAs fit on an SM when the ring stays near 100 KB: the next block's CTAs then become resident while
    // this block's finish, and fetch their first weight tiles meanwhile.
    const int ring_cap = 4 * stage_bytes <= 100 * 1024 ? 100 * 1024 : 200 * 1024;
    const int stages = std::max(1, std::min(nkb, ring_cap / stage_bytes));
    const int ring = std::max(stages * stage_bytes, 512 * Npad);
    const int smem = ring + 1024 + 256 + 16 * stages;
    int tmem_cols = 32;
    while (tmem_cols < Npad) tmem_cols *= 2;
    auto kern = KS == 4 ? head_swap_kernel<4> : head_swap_kernel<2>;
    static unsigned long long allowed[2] = {0, 0};                        // per device: large dynamic shared memory granted
    int dev = 0;
    cudaGetDevice(&dev);
    if (!((allowed[KS == 4] >> (dev & 63)) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);   // the opt-in limit less the static part
        if (e != cudaSuccess) return e;
        allowed[KS == 4] |= 1ull << (dev & 63);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((p.d / BM) * KS));
    cfg.blockDim = dim3(SW_THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)KS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may be placed while the previous kernel drains
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, mx, mw, p, Npad, stages, tmem_cols);
}

// Blocks [first, end) of the chain in one launch; cooperative when it spans more than one block (its CTAs
// then wait for one another's tiles and must all be resident).  PAIR: clusters of two CTAs, one 256-row tile each.
template <int BN, bool PAIR>
cudaError_t launch_chain(ChainParams& p, int first, int end, int sm_count, bool cooperative, cudaStream_t s) {
    using C = Cfg<BN, PAIR>;
    static unsigned long long allowed = 0;                                // per device: large dynamic shared memory granted
    int dev = 0;
    cudaGetDevice(&dev);
    if (!((allowed >> (dev & 63)) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(head_chain_kernel<BN, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
        if (e != cudaSuccess) return e;
        allowed |= 1ull << (dev & 63);
    }
    p.first = first;
    p.end = end;
    constexpr int TM = PAIR ? 2 * BM : BM;
    const int ntiles = (end - first) * (p.d / BN) * ((p.M + TM - 1) / TM);
    const int workers = std::min(ntiles, PAIR ? sm_count / 2 : sm_count);  // one CTA per SM (its ring fills the shared memory)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * workers : workers));
    cfg.blockDim = dim3(HEAD_THREADS);
    cfg.dynamicSmemBytes = (size_t)C::SMEM;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = cooperative ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = PAIR ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, head_chain_kernel<BN, PAIR>, p);
}

int fail(specdec_ctx* ctx, int code, const char* msg) {
    snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
    return code;
}

// One call of the head for more than 256 rows: all D blocks as tiles of one launch (`coop`) or one launch per block.
cudaError_t launch_chain_call(specdec_ctx* ctx, const __nv_bfloat16* x, const specdec_head* head, int M, int d, int D, int BN,
                              float* accept_prob, bool pair, bool coop, cudaStream_t s) {
    ChainParams p = {};
    for (int k = 0; k < D; ++k) {
        if (!cached_map(ctx, &p.mapX[k], x, M, d, BM) || !cached_map(ctx, &p.mapW[k], head->W[k], d, d, pair ? BN / 2 : BN))
            return cudaErrorUnknown;
        p.layer[k].X = x;
        p.layer[k].bias = static_cast<const __nv_bfloat16*>(head->b ? head->b[k] : nullptr);
        p.layer[k].Y = k == D - 1 ? nullptr : static_cast<__nv_bfloat16*>(ctx->act[k & 1]);
        if (p.layer[k].Y) {
            if (!cached_map(ctx, &p.mapY[k], p.layer[k].Y, M, d, OUT_ROWS, OUT_COLS)) return cudaErrorUnknown;
        } else {
            p.mapY[k] = p.mapX[0];
        }
        x = p.layer[k].Y;
    }
    for (int k = D; k < CHAIN_MAX; ++k) {                      // unused slots: defined bytes for the parameter copy
        p.mapX[k] = p.mapX[0];
        p.mapW[k] = p.mapW[0];
        p.mapY[k] = p.mapX[0];
        p.layer[k] = ChainLayer{nullptr, nullptr, nullptr};
    }
    p.depth = D;
    p.M = M;
    p.d = d;
    p.w_out = static_cast<const __nv_bfloat16*>(head->w_out);
    p.partial = ctx->head_partial;
    p.ready = ctx->head_ready + 1;
    p.exited = ctx->head_ready;
    p.accept_prob = accept_prob;
    p.b_out = head->b_out;
    p.status = ctx->status;
    auto launch = [&](int first, int end) {
        if (pair)
            return BN == 256 ? launch_chain<256, true>(p, first, end, ctx->sm_count, coop, s)
                             : launch_chain<128, true>(p, first, end, ctx->sm_count, coop, s);
        return BN == 256 ? launch_chain<256, false>(p, first, end, ctx->sm_count, coop, s)
                         : launch_chain<128, false>(p, first, end, ctx->sm_count, coop, s);
    };
    if (coop) {
        const cudaError_t e = launch(0, D);
        if (e != cudaSuccess) return e;
        ctx->launches += 1;
    } else {
        for (int k = 0; k < D; ++k) {
            const cudaError_t e = launch(k, k + 1);
            if (e != cudaSuccess) return e;             // after a first block was enqueued: a real error, not a refused configuration
            ctx->launches += 1;
        }
    }
    return cudaSuccess;
}


}  // namespace

#ifdef SPECDEC_STAMPS
// Diagnostic build only (not part of the public header): the phase timestamps of one CTA of the last two
// launches of the weights-as-M kernel, [block (0 first / 1 last)][warp][slot] in ns of the global timer.
extern "C" int specdec_debug_head_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, head_stamps, sizeof(head_stamps));
}
// The per-tile timestamps of the first and last CTA of the last launch of the 128-row-tile kernel.
extern "C" int specdec_debug_head_tile_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, head_tile_stamps, sizeof(head_tile_stamps));
}
#endif

extern "C" int specdec_accept_head(specdec_ctx* ctx, const void* hidden, const specdec_head* head, int B, int K,
                                   float* accept_prob, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!hidden || !head || !accept_prob || !head->w_out) return fail(ctx, SPECDEC_EINVAL, "accept_head: null pointer argument");
    if (B < 1 || K < 1) return fail(ctx, SPECDEC_EINVAL, "accept_head: B and K must be >= 1");
    const int d = head->d, D = head->depth;
    if (D < 0 || D > 8) return fail(ctx, SPECDEC_EINVAL, "accept_head: depth must be in [0, 8]");
    if (D > 0 && !head->W) return fail(ctx, SPECDEC_EINVAL, "accept_head: null weight list");
    if (d < 128 || d % 128 != 0) return fail(ctx, SPECDEC_EUNSUPPORTED, "accept_head: d must be a positive multiple of 128");
    const long long M = (long long)B * K;
    if (d > ctx->max_d || M > (long long)ctx->max_B * ctx->max_K)
        return fail(ctx, SPECDEC_EUNSUPPORTED, "accept_head: B*K or d exceed the context");
    if (reinterpret_cast<uintptr_t>(hidden) % 16 != 0 || reinterpret_cast<uintptr_t>(head->w_out) % 16 != 0)
        return fail(ctx, SPECDEC_EINVAL, "accept_head: hidden and w_out must be 16-byte aligned");
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(hidden);
    if (D == 0) {
        const int wpb = 8;
        head_linear_kernel<<<(int)((M + wpb - 1) / wpb), wpb * 32, 0, s>>>(x, static_cast<const __nv_bfloat16*>(head->w_out),
                                                                            (int)M, d, head->b_out, accept_prob);
        ctx->launches += 1;
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? SPECDEC_OK : fail(ctx, SPECDEC_ECUDA, cudaGetErrorString(e));
    }
    // Column tiles of 256 where the width allows, except when a block then has so few tiles that half the SMs
    // would idle (a tile is 256 rows: a pair of CTAs): 128-wide tiles take 0.7 of the time of 256-wide ones, so
    // they pay only there (measured at d = 4096: 512 rows 63.5 against 73.8 us, 768 rows 86.0 against 75.9 us).
    const long long wide_tiles = ((M + 2 * BM - 1) / (2 * BM)) * (d / 256);
    const int BN = d % 256 == 0 && wide_tiles * 4 > ctx->sm_count ? 256 : 128;
    // up to 256 rows: the weights as the M-side operand, N = the rows rounded up to 16
    const int Npad = (int)((M + 15) / 16 * 16);
    const bool swap_path = M <= 256;
    for (int k = 0; k < D; ++k) {
        const void* W = head->W[k];
        const void* bias = head->b ? head->b[k] : nullptr;
        if (!W || reinterpret_cast<uintptr_t>(W) % 16 != 0 || (bias && reinterpret_cast<uintptr_t>(bias) % 16 != 0))
            return fail(ctx, SPECDEC_EINVAL, "accept_head: weights and biases must be non-null and 16-byte aligned");
    }
    if (swap_path) {
        for (int k = 0; k < D; ++k) {
            const bool last = (k == D - 1);
            CUtensorMap mx, mw;
            if (!cached_map(ctx, &mx, x, (int)M, d, Npad) || !cached_map(ctx, &mw, head->W[k], d, d, BM))
                return fail(ctx, SPECDEC_ECUDA, "accept_head: cuTensorMapEncodeTiled failed");
            BlockParams p;
            p.X = x;
            p.bias = static_cast<const __nv_bfloat16*>(head->b ? head->b[k] : nullptr);
            p.Y = last ? nullptr : static_cast<__nv_bfloat16*>(ctx->act[k & 1]);
            p.w_out = last ? static_cast<const __nv_bfloat16*>(head->w_out) : nullptr;
            p.partial = last ? ctx->head_partial : nullptr;
            p.M = (int)M;
            p.d = d;
            p.status = ctx->status;
            p.done_ctr = ctx->task_ctl + 6;
            p.accept_prob = accept_prob;
            p.b_out = head->b_out;
            cudaError_t e = launch_swap(mx, mw, p, Npad, s);
            if (e != cudaSuccess) return fail(ctx, SPECDEC_ECUDA, cudaGetErrorString(e));
            ctx->launches += 1;
            x = p.Y;
        }
    } else {
        // Preferred: a pair of CTAs per 256-row tile (a third less operand traffic per SM) and all blocks in one
        // cooperative launch.  A device or partition that refuses clusters or the cooperative grid gets one CTA
        // per tile, then one launch per block; what was refused is remembered in the context.
        for (;;) {
            const bool pair = ctx->head_pair != 0 && ctx->sm_count >= 2;
            const bool coop = ctx->head_coop != 0 && D > 1;
            cudaError_t e = launch_chain_call(ctx, x, head, (int)M, d, D, BN, accept_prob, pair, coop, s);
            if (e == cudaSuccess) break;
            const bool config_error = e == cudaErrorCooperativeLaunchTooLarge || e == cudaErrorNotSupported ||
                                      e == cudaErrorInvalidValue || e == cudaErrorInvalidConfiguration ||
                                      e == cudaErrorLaunchOutOfResources;
            if (!config_error || (!pair && !coop)) return fail(ctx, SPECDEC_ECUDA, cudaGetErrorString(e));
            (void)cudaGetLastError();
            if (pair) ctx->head_pair = 0;
            else ctx->head_coop = 0;
        }
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SPECDEC_OK : fail(ctx, SPECDEC_ECUDA, cudaGetErrorString(e));
}
