// C ABI of libspecdec: context management, argument checks and dispatch to the launchers.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "specdec_internal.h"

namespace {

int fail(specdec_ctx* ctx, int code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

int cuda_fail(specdec_ctx* ctx, cudaError_t e, const char* what) {
    return fail(ctx, SPECDEC_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CU(ctx, call)                                              \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call); \
    } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_verify_args(specdec_ctx* ctx, const void* target, const void* draft, int dtype, const int32_t* tokens,
                      const float* uniforms, float T, int B, int K, int V, const int32_t* n_acc,
                      const int32_t* next, uint32_t flags) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!target || !draft || !tokens || !uniforms || !n_acc || !next)
        return fail(ctx, SPECDEC_EINVAL, "verify_correct: null pointer argument");
    if (dtype != SPECDEC_F32 && dtype != SPECDEC_BF16) return fail(ctx, SPECDEC_EINVAL, "verify_correct: unknown dtype %d", dtype);
    if (reinterpret_cast<uintptr_t>(target) % 4 != 0 || reinterpret_cast<uintptr_t>(draft) % 4 != 0)
        return fail(ctx, SPECDEC_EINVAL, "verify_correct: logit tensors must be 4-byte aligned");
    if (B < 1 || K < 1 || V < 1) return fail(ctx, SPECDEC_EINVAL, "verify_correct: B, K, V must be >= 1 (got %d, %d, %d)", B, K, V);
    if (!(T > 0.f) || !std::isfinite(T)) return fail(ctx, SPECDEC_EINVAL, "verify_correct: temperature must be positive and finite");
    if ((flags & ~SPECDEC_VERIFY_EARLY_EXIT) > SPECDEC_VERIFY_CLUSTER) return fail(ctx, SPECDEC_EINVAL, "verify_correct: unknown flags %u", flags);
    if (B > ctx->max_B || K > ctx->max_K)
        return fail(ctx, SPECDEC_EUNSUPPORTED, "verify_correct: B=%d K=%d exceed the context (max_B=%d max_K=%d)", B, K, ctx->max_B, ctx->max_K);
    if (V > (1 << 22)) return fail(ctx, SPECDEC_EUNSUPPORTED, "verify_correct: V=%d above 2^22", V);
    return specdec_use_device(ctx);
}

}  // namespace

// Every entry point runs on the context's GPU, whichever device the calling thread had current.
int specdec_use_device(specdec_ctx* ctx) {
    int cur = -1;
    if (cudaGetDevice(&cur) == cudaSuccess && cur == ctx->device) return SPECDEC_OK;   // the usual case, no driver call
    cudaError_t e = cudaSetDevice(ctx->device);
    return e == cudaSuccess ? SPECDEC_OK : cuda_fail(ctx, e, "cudaSetDevice");
}

extern "C" {

int specdec_create(specdec_ctx** out, int device, int max_B, int max_K, int max_d) {
    if (!out || max_B < 1 || max_K < 1 || max_d < 0 || device < 0) return SPECDEC_EINVAL;
    *out = nullptr;
    if ((long long)max_B * (max_K + 1) > (1ll << 28)) return SPECDEC_EINVAL;
    specdec_ctx* ctx = new (std::nothrow) specdec_ctx();
    if (!ctx) return SPECDEC_ECUDA;
    ctx->device = device;
    ctx->max_B = max_B;
    ctx->max_K = max_K;
    ctx->max_d = max_d;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    const size_t nflag = (size_t)max_B * max_K, ndraw = (size_t)max_B * (max_K + 1);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->flags, nflag * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->draws, ndraw * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->draw_mass, ndraw * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->arrive, (size_t)max_B * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->status, sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->early_exits, sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(ctx->early_exits, 0, sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->norms, ndraw * sizeof(float4));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->tasks, (size_t)max_B * sizeof(int2));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->task_ctl, 8 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->task_ctl, 0, 8 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->task_ready, (size_t)max_B * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->task_ready, 0, (size_t)max_B * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->flags, 0, nflag * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->arrive, 0, (size_t)max_B * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->status, 0, sizeof(uint32_t));
    if (e == cudaSuccess && max_d > 0) {
        const size_t act = (size_t)max_B * max_K * max_d * 2;
        e = cudaMalloc(&ctx->act[0], act);
        if (e == cudaSuccess) e = cudaMalloc(&ctx->act[1], act);
        if (e == cudaSuccess)
            e = cudaMalloc(&ctx->head_partial, (size_t)max_B * max_K * ((max_d + 31) / 32) * sizeof(float));
        if (e == cudaSuccess)
        {
            const size_t n = (1 + 8 * (((size_t)max_B * max_K + 127) / 128 + 1)) * sizeof(uint32_t);
            e = cudaMalloc(&ctx->head_ready, n);
            if (e == cudaSuccess) e = cudaMemset(ctx->head_ready, 0, n);
        }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        specdec_destroy(ctx);
        return SPECDEC_ECUDA;
    }
    *out = ctx;
    return SPECDEC_OK;
}

int specdec_destroy(specdec_ctx* ctx) {
    if (!ctx) return SPECDEC_EINVAL;
    cudaSetDevice(ctx->device);
    cudaFree(ctx->flags);
    cudaFree(ctx->draws);
    cudaFree(ctx->draw_mass);
    cudaFree(ctx->arrive);
    cudaFree(ctx->status);
    cudaFree(ctx->early_exits);
    cudaFree(ctx->norms);
    cudaFree(ctx->tasks);
    cudaFree(ctx->task_ctl);
    cudaFree(ctx->task_ready);
    cudaFree(ctx->stage);
    cudaFree(ctx->act[0]);
    cudaFree(ctx->act[1]);
    cudaFree(ctx->head_partial);
    cudaFree(ctx->head_ready);
    delete ctx;
    return SPECDEC_OK;
}

const char* specdec_last_error(const specdec_ctx* ctx) { return ctx ? ctx->err : "null context"; }

uint64_t specdec_launch_count(const specdec_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* specdec_last_kernel(const specdec_ctx* ctx) { return ctx ? ctx->last_kernel : "none"; }

int specdec_early_exit_count(specdec_ctx* ctx, void* stream, uint64_t* units) {
    if (!ctx || !units) return SPECDEC_EINVAL;
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned long long host = 0;
    CU(ctx, cudaMemcpyAsync(&host, ctx->early_exits, sizeof(host), cudaMemcpyDeviceToHost, s));
    CU(ctx, cudaMemsetAsync(ctx->early_exits, 0, sizeof(host), s));
    CU(ctx, cudaStreamSynchronize(s));
    *units = host;
    return SPECDEC_OK;
}

int specdec_set_phase_stamps(specdec_ctx* ctx, uint64_t* stamps, size_t units) {
    if (!ctx) return SPECDEC_EINVAL;
#ifdef SPECDEC_STAMPS
    ctx->stamps = reinterpret_cast<unsigned long long*>(stamps);
    ctx->stamps_units = stamps ? units : 0;
    return SPECDEC_OK;
#else
    (void)units;
    if (!stamps) return SPECDEC_OK;
    return fail(ctx, SPECDEC_EUNSUPPORTED, "set_phase_stamps: this build of the library carries no timestamp code (build with -DSPECDEC_STAMPS)");
#endif
}

int specdec_head_launch_mode(specdec_ctx* ctx, int pair, int cooperative) {
    if (!ctx) return SPECDEC_EINVAL;
    ctx->head_pair = pair ? 1 : 0;
    ctx->head_coop = cooperative ? -1 : 0;                 // -1: allowed, not yet confirmed by a launch
    return SPECDEC_OK;
}

int specdec_device_status(specdec_ctx* ctx, void* stream, uint32_t* bits) {
    if (!ctx) return SPECDEC_EINVAL;
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t host = 0;
    CU(ctx, cudaMemcpyAsync(&host, ctx->status, sizeof(host), cudaMemcpyDeviceToHost, s));
    CU(ctx, cudaMemsetAsync(ctx->status, 0, sizeof(uint32_t), s));
    CU(ctx, cudaStreamSynchronize(s));
    if (bits) *bits = host;
    if (host) return fail(ctx, SPECDEC_EDATA, "device status bits 0x%x (1 = bad cand_len, 2 = bad token, 4 = wait limit, 8 = top-k ties)", host);
    return SPECDEC_OK;
}

int specdec_verify_correct(specdec_ctx* ctx, const void* target_logits, const void* draft_logits,
                           specdec_dtype dtype, const int32_t* cand_tokens, const int32_t* cand_len,
                           const float* uniforms, float temperature, int B, int K, int V, int32_t* n_accepted,
                           int32_t* next_token, float* accept_ratio, float* row_stats, float* resid_mass,
                           uint32_t flags, void* stream) {
    int rc = check_verify_args(ctx, target_logits, draft_logits, (int)dtype, cand_tokens, uniforms, temperature, B,
                               K, V, n_accepted, next_token, flags);
    if (rc != SPECDEC_OK) return rc;
    if (row_stats && reinterpret_cast<uintptr_t>(row_stats) % 16 != 0)
        return fail(ctx, SPECDEC_EINVAL, "verify_correct: row_stats must be 16-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ctx->epoch = (ctx->epoch + 1) & 0x3fffffffu;
    if ((ctx->epoch & 0xffffffu) == 0)   // the row records carry 24 epoch bits
        CU(ctx, cudaMemsetAsync(ctx->task_ready, 0, (size_t)ctx->max_B * sizeof(int32_t), s));
    if (ctx->epoch == 0) {   // wrapped: forget every stale flag before reusing epoch numbers
        CU(ctx, cudaMemsetAsync(ctx->flags, 0, (size_t)ctx->max_B * ctx->max_K * sizeof(int32_t), s));
        ctx->epoch = 1;
    }
    VerifyParams p;
    p.target = target_logits;
    p.draft = draft_logits;
    p.tokens = cand_tokens;
    p.lens = cand_len;
    p.uniforms = uniforms;
    p.c = (float)(1.4426950408889634 / (double)temperature);
    p.B = B;
    p.K = K;
    p.V = V;
    p.n_acc = n_accepted;
    p.next = next_token;
    p.ratio = accept_ratio;
    p.stats = row_stats;
    p.rmass = resid_mass;
    p.flags = ctx->flags;
    p.draws = ctx->draws;
    p.draw_mass = ctx->draw_mass;
    p.arrive = ctx->arrive;
    p.status = ctx->status;
    p.norms = ctx->norms;
    p.tasks = ctx->tasks;
    p.task_ctl = ctx->task_ctl;
    p.task_ready = ctx->task_ready;
    p.epoch = ctx->epoch;
    if (ctx->stamps && (size_t)B * (K + 1) <= ctx->stamps_units) p.stamps = ctx->stamps;

    const bool stream_ok = verify_stream_supported(p, dtype);
    uint32_t kind = flags & ~SPECDEC_VERIFY_EARLY_EXIT;
    if ((flags & SPECDEC_VERIFY_EARLY_EXIT) && !accept_ratio && !row_stats) p.early_exits = ctx->early_exits;
    if (kind == SPECDEC_VERIFY_AUTO) {
        // One CTA per unit (four 256-thread CTAs per SM on large grids) measured at or ahead of the
        // persistent TMA pipelines at every size tried, so those stay selectable but are not picked here.
        // A handful of units: several CTAs per unit, each on a slice of the vocabulary.
        kind = verify_cluster_size(p, dtype, ctx->sm_count) > 1 ? SPECDEC_VERIFY_CLUSTER : SPECDEC_VERIFY_DIRECT;
    }
    if (kind == SPECDEC_VERIFY_FUSED && K > 63) kind = SPECDEC_VERIFY_STREAM;     // row records hold n in 6 bits
    if ((kind == SPECDEC_VERIFY_STREAM || kind == SPECDEC_VERIFY_FUSED) && !stream_ok)
        return fail(ctx, SPECDEC_EUNSUPPORTED, "verify_correct: streaming kernels need 16-byte aligned rows (V=%d)", V);
    int n_launch = 0;
    const int csize = kind == SPECDEC_VERIFY_CLUSTER ? verify_cluster_size(p, dtype, ctx->sm_count) : 1;
    cudaError_t e = kind == SPECDEC_VERIFY_CLUSTER  ? launch_verify_cluster(p, dtype, csize > 1 ? csize : 2, s, &n_launch)
                    : kind == SPECDEC_VERIFY_FUSED  ? launch_verify_fused(p, dtype, ctx->sm_count, s, &n_launch)
                    : kind == SPECDEC_VERIFY_STREAM ? launch_verify_stream(p, dtype, ctx->sm_count, s, &n_launch)
                                                    : launch_verify_direct(p, dtype, s, &n_launch);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "verify_correct launch");
    ctx->launches += n_launch;
    ctx->last_kernel = kind == SPECDEC_VERIFY_CLUSTER  ? "verify_cluster_kernel"
                       : kind == SPECDEC_VERIFY_FUSED  ? "verify_fused_kernel"
                       : kind == SPECDEC_VERIFY_STREAM ? "verify_stream_stats_kernel"
                                                       : "verify_direct_kernel";
    return SPECDEC_OK;
}

int specdec_verify_correct_topk(specdec_ctx* ctx, const void* target_logits, const void* draft_logits,
                                specdec_dtype dtype, const int32_t* cand_tokens, const int32_t* cand_len,
                                const float* uniforms, float temperature, int top_k, int B, int K, int V,
                                int32_t* n_accepted, int32_t* next_token, float* accept_ratio, float* resid_mass,
                                void* stream) {
    if (ctx && top_k >= V && V >= 1)
        return specdec_verify_correct(ctx, target_logits, draft_logits, dtype, cand_tokens, cand_len, uniforms,
                                      temperature, B, K, V, n_accepted, next_token, accept_ratio, nullptr,
                                      resid_mass, SPECDEC_VERIFY_AUTO, stream);
    int rc = check_verify_args(ctx, target_logits, draft_logits, (int)dtype, cand_tokens, uniforms, temperature, B,
                               K, V, n_accepted, next_token, SPECDEC_VERIFY_AUTO);
    if (rc != SPECDEC_OK) return rc;
    if (top_k < 1 || top_k > 256) return fail(ctx, SPECDEC_EINVAL, "verify_correct_topk: top_k must be in [1, 256] or >= V (got %d)", top_k);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ctx->epoch = (ctx->epoch + 1) & 0x3fffffffu;
    if ((ctx->epoch & 0xffffffu) == 0)
        CU(ctx, cudaMemsetAsync(ctx->task_ready, 0, (size_t)ctx->max_B * sizeof(int32_t), s));
    if (ctx->epoch == 0) {
        CU(ctx, cudaMemsetAsync(ctx->flags, 0, (size_t)ctx->max_B * ctx->max_K * sizeof(int32_t), s));
        ctx->epoch = 1;
    }
    VerifyParams p = {};
    p.target = target_logits;
    p.draft = draft_logits;
    p.tokens = cand_tokens;
    p.lens = cand_len;
    p.uniforms = uniforms;
    p.c = (float)(1.4426950408889634 / (double)temperature);
    p.B = B;
    p.K = K;
    p.V = V;
    p.n_acc = n_accepted;
    p.next = next_token;
    p.ratio = accept_ratio;
    p.rmass = resid_mass;
    p.flags = ctx->flags;
    p.draws = ctx->draws;
    p.draw_mass = ctx->draw_mass;
    p.arrive = ctx->arrive;
    p.status = ctx->status;
    p.epoch = ctx->epoch;
    cudaError_t e = launch_verify_topk(p, dtype, top_k, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "verify_correct_topk launch");
    ctx->launches += 1;
    ctx->last_kernel = "verify_topk_kernel";
    return SPECDEC_OK;
}

int specdec_sample(specdec_ctx* ctx, const void* logits, specdec_dtype dtype, const float* uniforms, float temperature,
                   int top_k, int B, int V, int32_t* tokens, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!logits || !uniforms || !tokens) return fail(ctx, SPECDEC_EINVAL, "sample: null pointer argument");
    if ((int)dtype != SPECDEC_F32 && (int)dtype != SPECDEC_BF16) return fail(ctx, SPECDEC_EINVAL, "sample: unknown dtype %d", (int)dtype);
    if (!(temperature > 0.f) || !std::isfinite(temperature)) return fail(ctx, SPECDEC_EINVAL, "sample: temperature must be positive and finite");
    if (reinterpret_cast<uintptr_t>(logits) % 4 != 0) return fail(ctx, SPECDEC_EINVAL, "sample: logits must be 4-byte aligned");
    if (V > (1 << 22)) return fail(ctx, SPECDEC_EUNSUPPORTED, "sample: V=%d above 2^22", V);
    if (B < 1 || V < 1) return fail(ctx, SPECDEC_EINVAL, "sample: B and V must be >= 1 (got %d, %d)", B, V);
    if (B > ctx->max_B) return fail(ctx, SPECDEC_EUNSUPPORTED, "sample: B=%d exceeds the context (max_B=%d)", B, ctx->max_B);
    if (top_k > 256 && top_k < V) return fail(ctx, SPECDEC_EINVAL, "sample: top_k must be <= 256, or <= 0 / >= V for none (got %d)", top_k);
    if (int rc0 = specdec_use_device(ctx)) return rc0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ctx->epoch = (ctx->epoch + 1) & 0x3fffffffu;
    if ((ctx->epoch & 0xffffffu) == 0)
        CU(ctx, cudaMemsetAsync(ctx->task_ready, 0, (size_t)ctx->max_B * sizeof(int32_t), s));
    if (ctx->epoch == 0) {
        CU(ctx, cudaMemsetAsync(ctx->flags, 0, (size_t)ctx->max_B * ctx->max_K * sizeof(int32_t), s));
        ctx->epoch = 1;
    }
    // Algorithm 2 with no candidates: every row is its own bonus position
    VerifyParams p = {};
    p.target = logits;
    p.draft = logits;
    p.uniforms = uniforms;
    p.c = (float)(1.4426950408889634 / (double)temperature);
    p.B = B;
    p.K = 0;
    p.V = V;
    p.n_acc = reinterpret_cast<int32_t*>(ctx->tasks);      // always 0 here; not reported
    p.next = tokens;
    p.flags = ctx->flags;
    p.draws = ctx->draws;
    p.draw_mass = ctx->draw_mass;
    p.arrive = ctx->arrive;
    p.status = ctx->status;
    p.norms = ctx->norms;
    p.tasks = ctx->tasks;
    p.task_ctl = ctx->task_ctl;
    p.task_ready = ctx->task_ready;
    p.epoch = ctx->epoch;
    int n_launch = 1;
    cudaError_t e = (top_k >= 1 && top_k < V) ? launch_verify_topk(p, dtype, top_k, s)
                                              : launch_verify_direct(p, dtype, s, &n_launch);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "sample launch");
    ctx->launches += n_launch;
    return SPECDEC_OK;
}

namespace {
int check_shard_args(specdec_ctx* ctx, const specdec_shard* sh, float T, int B, int K, const char* who) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!sh || !sh->target_logits || !sh->draft_logits) return fail(ctx, SPECDEC_EINVAL, "%s: null shard or logits", who);
    if ((int)sh->dtype != SPECDEC_F32 && (int)sh->dtype != SPECDEC_BF16) return fail(ctx, SPECDEC_EINVAL, "%s: unknown dtype %d", who, (int)sh->dtype);
    if (B < 1 || K < 1) return fail(ctx, SPECDEC_EINVAL, "%s: B and K must be >= 1 (got %d, %d)", who, B, K);
    if (sh->V_shard < 1 || sh->v_offset < 0 || sh->V < 1 || (long long)sh->v_offset + sh->V_shard > (long long)sh->V)
        return fail(ctx, SPECDEC_EINVAL, "%s: columns [%d, %d + %d) do not lie in a vocabulary of %d", who, sh->v_offset, sh->v_offset, sh->V_shard, sh->V);
    if (!(T > 0.f) || !std::isfinite(T)) return fail(ctx, SPECDEC_EINVAL, "%s: temperature must be positive and finite", who);
    if (sh->V > (1 << 22)) return fail(ctx, SPECDEC_EUNSUPPORTED, "%s: V=%d above 2^22", who, sh->V);
    return specdec_use_device(ctx);
}
}  // namespace

int specdec_shard_stats(specdec_ctx* ctx, const specdec_shard* shard, const int32_t* cand_tokens,
                        const int32_t* cand_len, float temperature, int B, int K, float* stats, void* stream) {
    int rc = check_shard_args(ctx, shard, temperature, B, K, "shard_stats");
    if (rc != SPECDEC_OK) return rc;
    if (!cand_tokens || !stats) return fail(ctx, SPECDEC_EINVAL, "shard_stats: null pointer argument");
    if (reinterpret_cast<uintptr_t>(stats) % 16 != 0) return fail(ctx, SPECDEC_EINVAL, "shard_stats: stats must be 16-byte aligned");
    const float c = (float)(1.4426950408889634 / (double)temperature);
    cudaError_t e = launch_shard_stats(*shard, cand_tokens, cand_len, c, B, K, stats, ctx->status, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "shard_stats launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

int specdec_shard_accept(specdec_ctx* ctx, const specdec_shard* shard, const float* stats_all, int n_shards,
                         const int32_t* cand_len, const float* uniforms, float temperature, int B, int K,
                         int32_t* n_accepted, float* accept_ratio, float* row_norm, double* mass, void* stream) {
    int rc = check_shard_args(ctx, shard, temperature, B, K, "shard_accept");
    if (rc != SPECDEC_OK) return rc;
    if (!stats_all || !uniforms || !n_accepted || !row_norm || !mass) return fail(ctx, SPECDEC_EINVAL, "shard_accept: null pointer argument");
    if (n_shards < 1 || n_shards > SPECDEC_SHARD_MAX_RANKS) return fail(ctx, SPECDEC_EINVAL, "shard_accept: n_shards must be in [1, %d] (got %d)", SPECDEC_SHARD_MAX_RANKS, n_shards);
    if (reinterpret_cast<uintptr_t>(stats_all) % 16 != 0 || reinterpret_cast<uintptr_t>(row_norm) % 16 != 0)
        return fail(ctx, SPECDEC_EINVAL, "shard_accept: stats_all and row_norm must be 16-byte aligned");
    const float c = (float)(1.4426950408889634 / (double)temperature);
    cudaError_t e = launch_shard_accept(*shard, stats_all, n_shards, cand_len, uniforms, c, B, K, n_accepted, accept_ratio,
                                        row_norm, mass, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "shard_accept launch");
    ctx->launches += 2;
    return SPECDEC_OK;
}

int specdec_shard_draw(specdec_ctx* ctx, const specdec_shard* shard, const float* stats_all, const double* mass_all,
                       int n_shards, int rank, const int32_t* n_accepted, const int32_t* cand_len,
                       const float* uniforms, const float* row_norm, float temperature, int B, int K,
                       int32_t* next_token, float* resid_mass, void* stream) {
    int rc = check_shard_args(ctx, shard, temperature, B, K, "shard_draw");
    if (rc != SPECDEC_OK) return rc;
    if (!stats_all || !mass_all || !n_accepted || !uniforms || !row_norm || !next_token)
        return fail(ctx, SPECDEC_EINVAL, "shard_draw: null pointer argument");
    if (n_shards < 1 || n_shards > SPECDEC_SHARD_MAX_RANKS || rank < 0 || rank >= n_shards)
        return fail(ctx, SPECDEC_EINVAL, "shard_draw: rank %d of %d shards (at most %d)", rank, n_shards, SPECDEC_SHARD_MAX_RANKS);
    if (reinterpret_cast<uintptr_t>(stats_all) % 16 != 0 || reinterpret_cast<uintptr_t>(row_norm) % 16 != 0)
        return fail(ctx, SPECDEC_EINVAL, "shard_draw: stats_all and row_norm must be 16-byte aligned");
    const float c = (float)(1.4426950408889634 / (double)temperature);
    cudaError_t e = launch_shard_draw(*shard, stats_all, mass_all, n_shards, rank, n_accepted, cand_len, uniforms, row_norm,
                                      c, B, K, next_token, resid_mass, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "shard_draw launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

int specdec_verify_greedy(specdec_ctx* ctx, const void* target_logits, specdec_dtype dtype,
                          const int32_t* cand_tokens, const int32_t* cand_len, int B, int K, int V,
                          int32_t* n_accepted, int32_t* next_token, int32_t* target_argmax, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!target_logits || !cand_tokens || !n_accepted || !next_token)
        return fail(ctx, SPECDEC_EINVAL, "verify_greedy: null pointer argument");
    if (dtype != SPECDEC_F32 && dtype != SPECDEC_BF16) return fail(ctx, SPECDEC_EINVAL, "verify_greedy: unknown dtype %d", (int)dtype);
    if (B < 1 || K < 1 || V < 1) return fail(ctx, SPECDEC_EINVAL, "verify_greedy: B, K, V must be >= 1");
    if (B > ctx->max_B || K > ctx->max_K)
        return fail(ctx, SPECDEC_EUNSUPPORTED, "verify_greedy: B=%d K=%d exceed the context (max_B=%d max_K=%d)", B, K, ctx->max_B, ctx->max_K);
    if (V > (1 << 22)) return fail(ctx, SPECDEC_EUNSUPPORTED, "verify_greedy: V=%d above 2^22", V);
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    ctx->epoch = (ctx->epoch + 1) & 0x3fffffffu;
    if ((ctx->epoch & 0xffffffu) == 0)
        CU(ctx, cudaMemsetAsync(ctx->task_ready, 0, (size_t)ctx->max_B * sizeof(int32_t), s));
    if (ctx->epoch == 0) {
        CU(ctx, cudaMemsetAsync(ctx->flags, 0, (size_t)ctx->max_B * ctx->max_K * sizeof(int32_t), s));
        ctx->epoch = 1;
    }
    VerifyParams p = {};
    p.target = target_logits;
    p.tokens = cand_tokens;
    p.lens = cand_len;
    p.B = B;
    p.K = K;
    p.V = V;
    p.n_acc = n_accepted;
    p.next = next_token;
    p.flags = ctx->flags;
    p.draws = ctx->draws;
    p.arrive = ctx->arrive;
    p.status = ctx->status;
    p.epoch = ctx->epoch;
    cudaError_t e = launch_greedy(p, dtype, target_argmax, s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "verify_greedy launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

int specdec_verify_correct_host(specdec_ctx* ctx, const void* target_logits, const void* draft_logits,
                                specdec_dtype dtype, const int32_t* cand_tokens, const int32_t* cand_len,
                                const float* uniforms, float temperature, int B, int K, int V,
                                int32_t* n_accepted, int32_t* next_token, float* accept_ratio, uint32_t flags,
                                void* stream) {
    int rc = check_verify_args(ctx, target_logits, draft_logits, (int)dtype, cand_tokens, uniforms, temperature, B,
                               K, V, n_accepted, next_token, flags);
    if (rc != SPECDEC_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t es = dtype == SPECDEC_BF16 ? 2 : 4;
    const size_t t_bytes = (size_t)B * (K + 1) * V * es, d_bytes = (size_t)B * K * V * es;
    const size_t tok_bytes = (size_t)B * K * 4, len_bytes = (size_t)B * 4, uni_bytes = (size_t)B * (K + 1) * 4;
    size_t off = 0;
    const size_t o_t = off;   off = align_up(off + t_bytes, 256);
    const size_t o_d = off;   off = align_up(off + d_bytes, 256);
    const size_t o_tok = off; off = align_up(off + tok_bytes, 256);
    const size_t o_len = off; off = align_up(off + len_bytes, 256);
    const size_t o_uni = off; off = align_up(off + uni_bytes, 256);
    const size_t o_n = off;   off = align_up(off + len_bytes, 256);
    const size_t o_nx = off;  off = align_up(off + len_bytes, 256);
    const size_t o_r = off;   off = align_up(off + tok_bytes, 256);
    if (off > ctx->stage_bytes) {
        CU(ctx, cudaStreamSynchronize(s));
        cudaFree(ctx->stage);
        ctx->stage = nullptr;
        ctx->stage_bytes = 0;
        CU(ctx, cudaMalloc(&ctx->stage, off));
        ctx->stage_bytes = off;
    }
    char* base = static_cast<char*>(ctx->stage);
    CU(ctx, cudaMemcpyAsync(base + o_t, target_logits, t_bytes, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(base + o_d, draft_logits, d_bytes, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(base + o_tok, cand_tokens, tok_bytes, cudaMemcpyHostToDevice, s));
    if (cand_len) CU(ctx, cudaMemcpyAsync(base + o_len, cand_len, len_bytes, cudaMemcpyHostToDevice, s));
    CU(ctx, cudaMemcpyAsync(base + o_uni, uniforms, uni_bytes, cudaMemcpyHostToDevice, s));
    rc = specdec_verify_correct(ctx, base + o_t, base + o_d, dtype, reinterpret_cast<int32_t*>(base + o_tok),
                                cand_len ? reinterpret_cast<int32_t*>(base + o_len) : nullptr,
                                reinterpret_cast<float*>(base + o_uni), temperature, B, K, V,
                                reinterpret_cast<int32_t*>(base + o_n), reinterpret_cast<int32_t*>(base + o_nx),
                                accept_ratio ? reinterpret_cast<float*>(base + o_r) : nullptr, nullptr, nullptr,
                                flags, s);
    if (rc != SPECDEC_OK) return rc;
    CU(ctx, cudaMemcpyAsync(n_accepted, base + o_n, len_bytes, cudaMemcpyDeviceToHost, s));
    CU(ctx, cudaMemcpyAsync(next_token, base + o_nx, len_bytes, cudaMemcpyDeviceToHost, s));
    if (accept_ratio) CU(ctx, cudaMemcpyAsync(accept_ratio, base + o_r, tok_bytes, cudaMemcpyDeviceToHost, s));
    CU(ctx, cudaStreamSynchronize(s));
    return SPECDEC_OK;
}

int specdec_stop(specdec_ctx* ctx, const float* accept_prob, const int32_t* cand_len, float h, int B, int K,
                 int32_t* stop_pos, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!accept_prob || !stop_pos) return fail(ctx, SPECDEC_EINVAL, "stop: null pointer argument");
    if (B < 1 || K < 1) return fail(ctx, SPECDEC_EINVAL, "stop: B and K must be >= 1");
    if (h != h) return fail(ctx, SPECDEC_EINVAL, "stop: threshold is NaN");
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaError_t e = launch_stop(accept_prob, cand_len, h, B, K, stop_pos, ctx->status, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "stop launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

int specdec_stop_step(specdec_ctx* ctx, const float* accept_prob_step, float* p_hat, float h, int B,
                      int32_t* stop, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (!accept_prob_step || !p_hat || !stop) return fail(ctx, SPECDEC_EINVAL, "stop_step: null pointer argument");
    if (B < 1) return fail(ctx, SPECDEC_EINVAL, "stop_step: B must be >= 1");
    if (h != h) return fail(ctx, SPECDEC_EINVAL, "stop_step: threshold is NaN");
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaError_t e = launch_stop_step(accept_prob_step, p_hat, h, B, stop, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "stop_step launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

int specdec_selftest_wait_limit(specdec_ctx* ctx, void* stream) {
    if (!ctx) return SPECDEC_EINVAL;
    if (int rc = specdec_use_device(ctx)) return rc;
    cudaError_t e = launch_wait_limit_selftest(ctx->status, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "selftest launch");
    ctx->launches += 1;
    return SPECDEC_OK;
}

}  // extern "C"
