// Verify/correct (Algorithm 2 of arXiv 2405.19715) on logits that arrive split along the
// vocabulary, the layout a tensor-parallel output layer leaves them in (the paper shards its 70B
// target over several GPUs, Appendix D.1).  Every rank holds columns [v_offset, v_offset + V_shard)
// of both models' logits for all rows; three local phases are separated by two small exchanges
// that the caller performs (all-gathers of B*(K+1)*8 floats and of B doubles per rank):
//
//   stats   per (row, position): running-sum statistics of the local columns, plus the drafted
//           token's two logits on the rank that holds that column;
//   accept  statistics of all ranks merged in rank order (the same arithmetic on every rank, so n
//           agrees bit for bit), accept tests, first rejection; then the local mass of the weights
//           y' is drawn from, (p - q)_+ or p, at position n;
//   draw    the rank whose column range contains the point u * W of the inverse CDF walks its own
//           columns; all others report -1.
//
// No kernel here waits for another launch or another GPU.
#include "verify_device.cuh"

namespace {

using namespace sd;

constexpr int SHARD_THREADS = 512;
constexpr int REC = SPECDEC_SHARD_STATS_WIDTH;     // floats per (row, position) record

struct ShardRows {
    const void* target;
    const void* draft;
    int Vs, v_offset, V;
};

template <typename T>
__device__ __forceinline__ const T* target_row(const ShardRows& S, int K, int b, int i) {
    return static_cast<const T*>(S.target) + ((size_t)b * (K + 1) + i) * (size_t)S.Vs;
}
template <typename T>
__device__ __forceinline__ const T* draft_row(const ShardRows& S, int K, int b, int i) {
    return static_cast<const T*>(S.draft) + ((size_t)b * K + i) * (size_t)S.Vs;
}

// ---- phase 1 -----------------------------------------------------------------------------
// record: {rs_p, s_p, rs_q, s_q, t_y, d_y, owned, 0}; t_y, d_y, owned are zero unless this rank
// holds column y, so that summing the records of all ranks yields them exactly.
// THREADS: 512, or 256 (four CTAs per SM) on grids that cover the machine many times over.
template <typename T, bool VEC, int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) shard_stats_kernel(ShardRows S, const int32_t* __restrict__ tokens,
                                                                    const int32_t* __restrict__ lens, float c, int B,
                                                                    int K, float* __restrict__ stats,
                                                                    uint32_t* __restrict__ status) {
    __shared__ Acc wp[THREADS / 32], wq[THREADS / 32];
    const int unit = blockIdx.x;
    const int i = unit / B, b = unit - i * B;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = lens ? lens[b] : K;
    float4* rec = reinterpret_cast<float4*>(stats + ((size_t)b * (K + 1) + i) * REC);
    if (L < 0 || L > K || i > L) {                   // nothing of this position is read
        if (tid == 0) {
            if ((L < 0 || L > K) && i == 0) atomicOr(status, SPECDEC_DATA_BAD_LENGTH);
            rec[0] = make_float4(NEG_BIG, 0.f, NEG_BIG, 0.f);
            rec[1] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        return;
    }
    const bool bonus = (i == L);
    const T* trow = target_row<T>(S, K, b, i);
    const T* drow = bonus ? trow : draft_row<T>(S, K, b, i);
    float t_y = 0.f, d_y = 0.f, owned = 0.f;
    if (tid == 0 && !bonus) {
        const int y = tokens[(size_t)b * K + i];
        if (y < 0 || y >= S.V) atomicOr(status, SPECDEC_DATA_BAD_TOKEN);
        else if (y >= S.v_offset && y < S.v_offset + S.Vs) {
            t_y = to_float(trow[y - S.v_offset]);
            d_y = to_float(drow[y - S.v_offset]);
            owned = 1.f;
        }
    }
    Acc ap = acc_init(), aq = acc_init();
    unit_stats<T, VEC, THREADS>(trow, drow, S.Vs, c, bonus, tid, ap, aq);
    ap = warp_merge(ap);
    aq = warp_merge(aq);
    if (lane == 0) { wp[warp] = ap; wq[warp] = aq; }
    __syncthreads();
    if (warp == 0) {
        constexpr int NW = THREADS / 32;
        Acc a = lane < NW ? wp[lane] : acc_init(), q = lane < NW ? wq[lane] : acc_init();
        a = warp_merge(a);
        q = warp_merge(q);
        if (lane == 0) {
            rec[0] = make_float4(a.rs, a.s, bonus ? NEG_BIG : q.rs, bonus ? 0.f : q.s);
            rec[1] = make_float4(t_y, d_y, owned, 0.f);
        }
    }
}

// ---- phase 2a: merged statistics, accept tests, first rejection (one warp per row) ---------
struct Merged {
    Acc p, q;
    float t_y, d_y, owned;
};
__device__ __forceinline__ Merged merge_records(const float* __restrict__ stats_all, int n_shards, int B, int K, int b,
                                                int i) {
    Merged m{acc_init(), acc_init(), 0.f, 0.f, 0.f};
    for (int r = 0; r < n_shards; ++r) {             // rank order: identical on every rank
        const float4* rec = reinterpret_cast<const float4*>(stats_all + (((size_t)r * B + b) * (K + 1) + i) * REC);
        const float4 a = rec[0], t = rec[1];
        m.p = acc_merge(m.p, Acc{a.x, a.y});
        m.q = acc_merge(m.q, Acc{a.z, a.w});
        m.t_y += t.x;
        m.d_y += t.y;
        m.owned += t.z;
    }
    return m;
}

__global__ void __launch_bounds__(32) shard_accept_kernel(const float* __restrict__ stats_all, int n_shards,
                                                          const int32_t* __restrict__ lens,
                                                          const float* __restrict__ uniforms, float c, int B, int K,
                                                          int32_t* __restrict__ n_acc, float* __restrict__ ratio_out,
                                                          float* __restrict__ row_norm) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int L = lens ? lens[b] : K;
    float4* norm_out = reinterpret_cast<float4*>(row_norm) + b;
    if (L < 0 || L > K) {
        if (lane == 0) { n_acc[b] = -1; *norm_out = make_float4(0.f, 0.f, 0.f, 0.f); }
        if (ratio_out) for (int j = lane; j < K; j += 32) ratio_out[(size_t)b * K + j] = 0.f;
        return;
    }
    int n = L, bad = 0;
    for (int i0 = 0; i0 < L; i0 += 32) {
        const int i = i0 + lane;
        int state = FLAG_ACCEPT;
        if (i < L) {
            const Merged m = merge_records(stats_all, n_shards, B, K, b, i);
            const float lp = fmaf(m.t_y, c, -m.p.rs) - log2f(m.p.s);
            const float lq = fmaf(m.d_y, c, -m.q.rs) - log2f(m.q.s);
            const float ratio = ratio_from_logs(lp, lq);
            const bool ok = m.owned == 1.f;          // exactly one rank held column y
            const float r = uniforms[(size_t)b * (K + 1) + i];
            state = !ok ? FLAG_BAD : (r >= ratio ? FLAG_REJECT : FLAG_ACCEPT);     // r == ratio rejects
            if (ratio_out) ratio_out[(size_t)b * K + i] = ok ? fminf(1.f, ratio) : -1.f;
        }
        const unsigned rej = __ballot_sync(0xffffffffu, state >= FLAG_REJECT);
        const unsigned bd = __ballot_sync(0xffffffffu, state == FLAG_BAD);
        if (rej && n == L) n = i0 + __ffs(rej) - 1;
        bad |= (bd != 0);
    }
    if (ratio_out) for (int j = L + lane; j < K; j += 32) ratio_out[(size_t)b * K + j] = 0.f;
    if (lane == 0) {
        if (bad) {
            n_acc[b] = -1;
            *norm_out = make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            const Merged m = merge_records(stats_all, n_shards, B, K, b, n);
            const Norm np = make_norm(m.p), nq = n < L ? make_norm(m.q) : np;
            n_acc[b] = n;
            *norm_out = make_float4(np.rs, np.inv, nq.rs, nq.inv);
        }
    }
}

// ---- phase 2b / 3: the local weights of position n --------------------------------------------
// One CTA per row.  WALK = false: only the local mass (fp64 sum of fp32 slab sums).  WALK = true:
// the owning rank walks its columns to the local point tau of the inverse CDF.
template <typename T, bool VEC, bool WALK>
__global__ void __launch_bounds__(SHARD_THREADS) shard_draw_kernel(
    ShardRows S, const int32_t* __restrict__ n_acc, const int32_t* __restrict__ lens,
    const float* __restrict__ row_norm, const float* __restrict__ stats_all, const double* __restrict__ mass_all,
    int n_shards, int rank, const float* __restrict__ uniforms, float c, int B, int K, double* __restrict__ mass_out,
    int32_t* __restrict__ next, float* __restrict__ rmass) {
    extern __shared__ float slab_sum[];
    __shared__ UnitShared sh;
    __shared__ int s_mode;
    __shared__ double s_tau;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int n = n_acc[b];
    const int L = lens ? lens[b] : K;
    if (n < 0) {                                     // bad row
        if (tid == 0) {
            if constexpr (WALK) { next[b] = -1; if (rmass) rmass[b] = 0.f; }
            else mass_out[b] = 0.0;
        }
        return;
    }
    int mode = n == L ? 2 : 1;
    const float4 nr = reinterpret_cast<const float4*>(row_norm)[b];
    if (tid == 0) { sh.np = Norm{nr.x, nr.y}; sh.nq = Norm{nr.z, nr.w}; }
    double tau = -1.0;
    if constexpr (WALK) {
        if (tid == 0) {
            // total mass and the rank that holds u * W, from the gathered local masses (rank order)
            double mr[SPECDEC_SHARD_MAX_RANKS];
            double W = 0.0;
            for (int r = 0; r < n_shards; ++r) { mr[r] = mass_all[(size_t)r * B + b]; W += mr[r]; }
            const double W_report = W;
            int md = mode;
            if (md == 1 && !(W > 1e-30)) {
                // p == q to rounding: draw from p itself; the target's local masses follow from the
                // statistics, s_r * 2^(rs_r - log2 Z)
                md = 2;
                W = 0.0;
                for (int r = 0; r < n_shards; ++r) {
                    const float4 a = *reinterpret_cast<const float4*>(stats_all + (((size_t)r * B + b) * (K + 1) + n) * REC);
                    mr[r] = (double)a.y * exp2((double)a.x - (double)nr.x - (double)nr.y);
                    W += mr[r];
                }
            }
            const double thr = (double)uniforms[(size_t)b * (K + 1) + K] * W;
            int owner = -1, lastpos = -1;
            double before = 0.0, run = 0.0;
            for (int r = 0; r < n_shards; ++r) {
                if (mr[r] > 0.0) lastpos = r;
                if (owner < 0 && run + mr[r] > thr) { owner = r; before = run; }
                run += mr[r];
            }
            if (owner < 0) {                         // rounding left nothing above u * W
                owner = lastpos < 0 ? 0 : lastpos;
                before = 0.0;
                for (int r = 0; r < owner; ++r) before += mr[r];
            }
            const double t = thr - before;
            s_mode = owner == rank ? md : 0;
            s_tau = t < 0.0 ? 0.0 : t;
            if (owner != rank) next[b] = -1;
            if (rmass) rmass[b] = mode == 2 ? 1.f : (float)W_report;
        }
        __syncthreads();
        mode = s_mode;
        tau = s_tau;
        if (mode == 0) return;                       // another rank draws this row
    } else {
        __syncthreads();
    }
    const T* trow = target_row<T>(S, K, b, n);
    const T* drow = mode == 1 ? draft_row<T>(S, K, b, n) : trow;
    VerifyParams P = {};
    P.V = S.Vs;
    P.c = c;
    unit_draw<T, VEC>(P, trow, drow, mode, 0.f, sh, slab_sum, tid, SHARD_THREADS, 0, tau);
    if (tid == 0) {
        if constexpr (WALK) next[b] = S.v_offset + sh.token;
        else mass_out[b] = sh.total;
    }
}

template <typename T>
bool shard_vec(const specdec_shard& sh) {
    constexpr int N = Elem<T>::EPV;
    return sh.V_shard % N == 0 && reinterpret_cast<uintptr_t>(sh.target_logits) % 16 == 0 &&
           reinterpret_cast<uintptr_t>(sh.draft_logits) % 16 == 0;
}
template <typename T>
size_t slab_bytes(int Vs) {
    constexpr int N = Elem<T>::EPV;
    const int nvec = (Vs + N - 1) / N;
    return (size_t)((nvec + 31) / 32) * sizeof(float);
}

template <typename T, bool WALK>
cudaError_t launch_draw_t(const specdec_shard& sh, const ShardRows& S, const int32_t* n_acc, const int32_t* lens,
                          const float* row_norm, const float* stats_all, const double* mass_all, int n_shards,
                          int rank, const float* uniforms, float c, int B, int K, double* mass_out, int32_t* next,
                          float* rmass, cudaStream_t s) {
    const size_t smem = slab_bytes<T>(sh.V_shard);
    auto kern = shard_vec<T>(sh) ? shard_draw_kernel<T, true, WALK> : shard_draw_kernel<T, false, WALK>;
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    kern<<<B, SHARD_THREADS, smem, s>>>(S, n_acc, lens, row_norm, stats_all, mass_all, n_shards, rank, uniforms, c, B,
                                        K, mass_out, next, rmass);
    return cudaGetLastError();
}

ShardRows rows_of(const specdec_shard& sh) {
    return ShardRows{sh.target_logits, sh.draft_logits, sh.V_shard, sh.v_offset, sh.V};
}

}  // namespace

template <typename T>
void launch_stats_t(const specdec_shard& sh, const ShardRows& S, const int32_t* tokens, const int32_t* lens, float c,
                    int B, int K, float* stats, uint32_t* status, cudaStream_t s) {
    const int grid = B * (K + 1);
    const bool vec = shard_vec<T>(sh), small = grid >= 12 * 148;
    if (small) {
        if (vec) shard_stats_kernel<T, true, 256><<<grid, 256, 0, s>>>(S, tokens, lens, c, B, K, stats, status);
        else shard_stats_kernel<T, false, 256><<<grid, 256, 0, s>>>(S, tokens, lens, c, B, K, stats, status);
    } else {
        if (vec) shard_stats_kernel<T, true, 512><<<grid, 512, 0, s>>>(S, tokens, lens, c, B, K, stats, status);
        else shard_stats_kernel<T, false, 512><<<grid, 512, 0, s>>>(S, tokens, lens, c, B, K, stats, status);
    }
}

cudaError_t launch_shard_stats(const specdec_shard& sh, const int32_t* tokens, const int32_t* lens, float c, int B,
                               int K, float* stats, uint32_t* status, cudaStream_t s) {
    const ShardRows S = rows_of(sh);
    if (sh.dtype == SPECDEC_BF16) launch_stats_t<__nv_bfloat16>(sh, S, tokens, lens, c, B, K, stats, status, s);
    else launch_stats_t<float>(sh, S, tokens, lens, c, B, K, stats, status, s);
    return cudaGetLastError();
}

cudaError_t launch_shard_accept(const specdec_shard& sh, const float* stats_all, int n_shards, const int32_t* lens,
                                const float* uniforms, float c, int B, int K, int32_t* n_acc, float* ratio,
                                float* row_norm, double* mass, cudaStream_t s) {
    shard_accept_kernel<<<B, 32, 0, s>>>(stats_all, n_shards, lens, uniforms, c, B, K, n_acc, ratio, row_norm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const ShardRows S = rows_of(sh);
    return sh.dtype == SPECDEC_BF16
               ? launch_draw_t<__nv_bfloat16, false>(sh, S, n_acc, lens, row_norm, stats_all, nullptr, n_shards, 0,
                                                     uniforms, c, B, K, mass, nullptr, nullptr, s)
               : launch_draw_t<float, false>(sh, S, n_acc, lens, row_norm, stats_all, nullptr, n_shards, 0, uniforms, c,
                                             B, K, mass, nullptr, nullptr, s);
}

cudaError_t launch_shard_draw(const specdec_shard& sh, const float* stats_all, const double* mass_all, int n_shards,
                              int rank, const int32_t* n_acc, const int32_t* lens, const float* uniforms,
                              const float* row_norm, float c, int B, int K, int32_t* next, float* rmass,
                              cudaStream_t s) {
    const ShardRows S = rows_of(sh);
    return sh.dtype == SPECDEC_BF16
               ? launch_draw_t<__nv_bfloat16, true>(sh, S, n_acc, lens, row_norm, stats_all, mass_all, n_shards, rank,
                                                    uniforms, c, B, K, nullptr, next, rmass, s)
               : launch_draw_t<float, true>(sh, S, n_acc, lens, row_norm, stats_all, mass_all, n_shards, rank, uniforms,
                                            c, B, K, nullptr, next, rmass, s);
}
