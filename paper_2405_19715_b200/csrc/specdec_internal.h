// Internal declarations shared by the translation units of libspecdec (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "specdec.h"

// A tensor map (TMA descriptor) the acceptance head has built, kept so that a repeated call with the same
// operand does not pay the driver's encoding again.
struct HeadMapEntry {
    const void* ptr = nullptr;
    int rows = 0, cols = 0, box_rows = 0, box_cols = 0;
    alignas(64) unsigned char map[128];
};

struct specdec_ctx {
    int device = 0;
    int max_B = 0, max_K = 0, max_d = 0;
    int sm_count = 0;
    // verify/correct scratch (device)
    int32_t* flags = nullptr;     // [max_B * max_K]      (epoch << 2) | state of each accept test
    int32_t* draws = nullptr;     // [max_B * (max_K+1)]  candidate y' drawn at each position
    float* draw_mass = nullptr;   // [max_B * (max_K+1)]  mass of the weights that draw came from
    int32_t* arrive = nullptr;    // [max_B]              positions of a row that have finished
    uint32_t* status = nullptr;   // sticky SPECDEC_DATA_* bits
    unsigned long long* early_exits = nullptr;   // logit rows not read by units that left early (SPECDEC_VERIFY_EARLY_EXIT) since last read
    float4* norms = nullptr;      // [max_B * (max_K+1)]  log2 normalisers {hi_p, lo_p, hi_q, lo_q} per position
    int2* tasks = nullptr;        // [max_B]              rows whose y' is still to be drawn: {b, n}
    int32_t* task_ctl = nullptr;  // [8]                  two-launch path: {tasks, finished CTAs}; fused path: {-, -, -, head, finished}; [6]: CTAs done in the last block of the weights-as-M head kernel
    int32_t* task_ready = nullptr;// [max_B]              fused path: record {epoch:24, mode:2, n:6} of each resolved row
    uint32_t epoch = 0;
    uint64_t launches = 0;
    const char* last_kernel = "none";   // name of the kernel the last verify/correct call launched
    unsigned long long* stamps = nullptr;   // caller's phase-timestamp buffer (diagnostic builds), or null
    size_t stamps_units = 0;                // (row, position) units it has room for
    // staging for the host-buffer entry point (device), grown on demand
    void* stage = nullptr;
    size_t stage_bytes = 0;
    // acceptance-head activations (device, bf16) and split-N partial logits
    void* act[2] = {nullptr, nullptr};   // [max_B*max_K, max_d] each
    float* head_partial = nullptr;       // [max_B*max_K, max_d/32]
    uint32_t* head_ready = nullptr;      // [0]: CTAs of the head launch that have left; then [8][ceil(max_B*max_K / 128) + 1] finished
                                         // epilogue warps per (block, 128-row block); all zero between launches (the kernel clears them)
    int head_pair = 1;                   // a pair of CTAs per 256-row tile (0: one CTA per 128-row tile)
    int head_coop = -1;                  // one cooperative launch for all blocks: 0 ruled out or refused (one launch per block)
    HeadMapEntry head_maps[32];          // round-robin cache, keyed by (pointer, rows, cols, box rows, box cols)
    int head_map_next = 0;
    char err[256] = "no error";
};

struct VerifyParams {
    const void* target;
    const void* draft;
    const int32_t* tokens;
    const int32_t* lens;
    const float* uniforms;
    float c;              // log2(e) / T: logits are scaled into base-2 exponents
    int B, K, V;
    int32_t* n_acc;
    int32_t* next;
    float* ratio;
    float* stats;
    float* rmass;
    int32_t* flags;
    int32_t* draws;
    float* draw_mass;
    int32_t* arrive;
    uint32_t* status;
    float4* norms;
    int2* tasks;
    int32_t* task_ctl;
    int32_t* task_ready;
    uint32_t epoch;
    unsigned long long* early_exits = nullptr;   // non-null: units after a row's known first rejection read nothing
    unsigned long long* stamps = nullptr;   // phase timestamps, SPECDEC_STAMP_SLOTS {globaltimer ns, SM clock} pairs per unit (diagnostic builds)
};



// Makes the context's GPU the calling thread's current device (api.cu); SPECDEC_OK or SPECDEC_ECUDA.
int specdec_use_device(specdec_ctx* ctx);

// Launchers (verify.cu, verify_stream.cu, stop.cu, head.cu).  Return a cudaError_t.
cudaError_t launch_verify_direct(const VerifyParams& p, specdec_dtype dtype, cudaStream_t s, int* n_launch);
cudaError_t launch_verify_stream(const VerifyParams& p, specdec_dtype dtype, int sm_count, cudaStream_t s,
                                 int* n_launch);
cudaError_t launch_verify_fused(const VerifyParams& p, specdec_dtype dtype, int sm_count, cudaStream_t s,
                                int* n_launch);
bool verify_stream_supported(const VerifyParams& p, specdec_dtype dtype);
cudaError_t launch_greedy(const VerifyParams& p, specdec_dtype dtype, int32_t* argmax_out, cudaStream_t s);
cudaError_t launch_stop(const float* accept_prob, const int32_t* lens, float h, int B, int K,
                        int32_t* stop_pos, uint32_t* status, cudaStream_t s);
cudaError_t launch_stop_step(const float* accept_prob_step, float* p_hat, float h, int B, int32_t* stop,
                             cudaStream_t s);
cudaError_t launch_wait_limit_selftest(uint32_t* status, cudaStream_t s);
cudaError_t launch_verify_topk(const VerifyParams& p, specdec_dtype dtype, int top_k, cudaStream_t s);
cudaError_t launch_shard_stats(const specdec_shard& sh, const int32_t* tokens, const int32_t* lens, float c, int B,
                               int K, float* stats, uint32_t* status, cudaStream_t s);
cudaError_t launch_shard_accept(const specdec_shard& sh, const float* stats_all, int n_shards, const int32_t* lens,
                                const float* uniforms, float c, int B, int K, int32_t* n_acc, float* ratio,
                                float* row_norm, double* mass, cudaStream_t s);
cudaError_t launch_shard_draw(const specdec_shard& sh, const float* stats_all, const double* mass_all, int n_shards,
                              int rank, const int32_t* n_acc, const int32_t* lens, const float* uniforms,
                              const float* row_norm, float c, int B, int K, int32_t* next, float* rmass,
                              cudaStream_t s);
// Cluster size the small-batch kernel would use for this problem (1: not worth it).
int verify_cluster_size(const VerifyParams& p, specdec_dtype dtype, int sm_count);
cudaError_t launch_verify_cluster(const VerifyParams& p, specdec_dtype dtype, int C, cudaStream_t s, int* n_launch);
