/*
 * specdec.h -- C ABI of the SpecDec++ verify/correct + adaptive-stop library (sm_100a).
 *
 * Operations follow arXiv 2405.19715:
 *   - verify/correct: Algorithm 2 and the lower half of Algorithm 1 (accept test
 *     r_i < p_i(y_i)/q_i(y_i), first rejection n, residual draw from Norm[(p-q)_+],
 *     bonus draw from p_{K+1}); the rejection step itself is Appendix C.
 *   - acceptance head: Eq. 3, sigmoid(f_theta(e_i)), with f_theta the (D+1)-layer
 *     SiLU ResNet of Section 5.1.
 *   - stop rule: Section 4.3 and the loop of Algorithm 1 (stop when
 *     1 - prod_i sigmoid(f_theta(e_i)) > h).
 *
 * Conventions
 *   - Every pointer marked "dev" is device memory of the context's GPU, owned by the
 *     caller, neither retained nor freed by the library.  "host" pointers are ordinary
 *     (preferably pinned) host memory.
 *   - Tensors are dense row-major with the last index fastest; logit tensors start on a 4-byte boundary
 *     (16-byte boundaries and rows of whole 16-byte vectors take the vectorised paths).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) unless stated otherwise; outputs are valid once the
 *     stream has been synchronised.
 *   - Every call that takes a context makes that context's GPU the calling thread's current
 *     device (cudaSetDevice) and leaves it so; a process that drives several GPUs creates one
 *     context per GPU.
 *   - A context owns small scratch buffers.  Two calls that use the same context must
 *     not overlap on the GPU (use one context per stream).
 *   - Return value: SPECDEC_OK or an error code; specdec_last_error() gives a message.
 *     Problems that only the device can see (a token outside [0,V), a length outside
 *     [0,K]) never trap: the row's outputs become -1 and a sticky status word is set,
 *     to be read with specdec_device_status().
 */
#ifndef SPECDEC_H_
#define SPECDEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct specdec_ctx specdec_ctx;

typedef enum { SPECDEC_F32 = 0, SPECDEC_BF16 = 1 } specdec_dtype;

typedef enum {
    SPECDEC_OK = 0,
    SPECDEC_EINVAL = 1,       /* bad host-visible argument                              */
    SPECDEC_EUNSUPPORTED = 2, /* shape exceeds what the context / kernels were sized for */
    SPECDEC_ECUDA = 3,        /* a CUDA runtime call failed                              */
    SPECDEC_EDATA = 4         /* the device met a bad token or candidate length          */
} specdec_status;

/* Bits of the device status word returned by specdec_device_status(). */
#define SPECDEC_DATA_BAD_LENGTH 1u /* some cand_len[b] outside [0,K]                     */
#define SPECDEC_DATA_BAD_TOKEN  2u /* some cand_tokens[b,i] outside [0,V)                */
#define SPECDEC_DATA_WAIT_LIMIT 4u /* a bounded in-kernel wait gave up (outputs invalid) */
#define SPECDEC_DATA_TOPK_TIES  8u /* top-k: thousands of logits tie with a row's k-th largest    */

/* Kernel selection for specdec_verify_correct (flags argument). 0 lets the library pick. */
#define SPECDEC_VERIFY_AUTO    0u
#define SPECDEC_VERIFY_DIRECT  1u /* one CTA per (row, position), plain global loads      */
#define SPECDEC_VERIFY_STREAM  2u /* persistent CTAs fed by bulk async copies (TMA): one launch for the
                                    statistics and accept tests, a second for the draws           */
#define SPECDEC_VERIFY_FUSED   3u /* the same pipeline in one launch: CTAs that run out of units
                                    stream the draws of rows that are already resolved.  Its CTAs
                                    wait (bounded) for rows resolved by other CTAs of the launch, so
                                    it needs the GPU to itself: if another process or stream keeps
                                    some of its CTAs from being resident, waits can run out, the
                                    call reports SPECDEC_DATA_WAIT_LIMIT and its outputs are invalid */
#define SPECDEC_VERIFY_CLUSTER 4u /* small batches: a cluster of 2-8 CTAs per (row, position), each taking
                                    a slice of the vocabulary, combined through distributed shared
                                    memory; picked automatically while the units fit the SMs twice   */

/* May be OR-ed into the kernel selection (honoured by the one-CTA-per-unit kernel, i.e. by SPECDEC_VERIFY_AUTO on
 * all but the smallest problems and by SPECDEC_VERIFY_DIRECT; ignored when accept_ratio or row_stats is requested):
 * a (row, position) unit that finds, when it starts, that an earlier position of its row has already been rejected
 * in this call reads no logits -- positions after the first rejection cannot change n_accepted or next_token
 * (Algorithm 2 takes the minimum over the rejected positions).  Units are scheduled earliest position first, so
 * on batches of several waves most units after a row's first rejection leave at once.  Drafted tokens are still
 * range-checked at every position; outputs are identical with and without the bit. */
#define SPECDEC_VERIFY_EARLY_EXIT 0x100u

/*
 * Create a context on `device` able to serve calls with B <= max_B and K <= max_K.
 * Allocates the scratch used by verify/correct (per-(row,position) flags and draws,
 * per-row arrival counters) and, when max_d > 0, the activation buffers of the
 * acceptance head for max_B*max_K tokens of width max_d.  Ownership of *out passes to
 * the caller (release with specdec_destroy).  Errors: EINVAL (null/negative), ECUDA.
 */
int specdec_create(specdec_ctx** out, int device, int max_B, int max_K, int max_d);
int specdec_destroy(specdec_ctx* ctx);

/* Message of the last error returned for this context (never NULL). */
const char* specdec_last_error(const specdec_ctx* ctx);

/*
 * Synchronise `stream`, read and clear the sticky device status word.  *bits receives the
 * SPECDEC_DATA_* bits (may be NULL).  Returns SPECDEC_OK if no bit was set, else SPECDEC_EDATA.
 */
int specdec_device_status(specdec_ctx* ctx, void* stream, uint32_t* bits);

/* Number of kernels this context has launched so far (for launch accounting). */
uint64_t specdec_launch_count(const specdec_ctx* ctx);

/* How specdec_accept_head launches the residual blocks (Eq. 3) when B*K > 256.  By default the call tries, and
 * remembers per context what the device accepted: a pair of CTAs (thread-block cluster of two) per 256-row tile
 * and all blocks in one cooperative launch; without clusters one CTA per 128-row tile; without a cooperative
 * grid one launch per block.  pair = 0 / cooperative = 0 rule the respective form out for this context from now
 * on (a partition on which it should not be tried; tests of the fallbacks); 1 allows it again.  Results are the
 * same in every form up to the summation order inside a tile, which does not change.  Host only; no GPU work. */
int specdec_head_launch_mode(specdec_ctx* ctx, int pair, int cooperative);

/* Synchronises `stream`; *logit_rows receives the number of logit rows (V elements each: two per candidate
 * position, one for a bonus position) that units leaving early under SPECDEC_VERIFY_EARLY_EXIT did not read
 * since the last call of this function (the counter is then cleared). */
int specdec_early_exit_count(specdec_ctx* ctx, void* stream, uint64_t* logit_rows);

/* Name of the kernel the last specdec_verify_correct / _topk call on this context launched (which
 * one SPECDEC_VERIFY_AUTO picked): a static string, "none" before the first call. */
const char* specdec_last_kernel(const specdec_ctx* ctx);

/*
 * Diagnostic (no counterpart in the paper): phase timestamps of the one-CTA-per-unit verify/correct
 * kernel.  Only a library compiled with -DSPECDEC_STAMPS contains the code; any other build returns
 * SPECDEC_EUNSUPPORTED for a non-NULL buffer.  After this call every specdec_verify_correct on the
 * context whose B*(K+1) <= units makes each (row, position) unit u = i*B + b write
 * SPECDEC_STAMP_SLOTS pairs {globaltimer in ns, SM cycle counter} at stamps[(u*SLOTS + slot)*2]:
 * slot 0 CTA started, 1 candidate length known, 10 scalar operands requested, 2 first thread's share of
 * the statistics pass done, 3 CTA-wide merge done, 4 accept test and draw decision taken, 5 decision
 * seen by all threads (11-13 inside the accept test: warps' sums merged, ratio formed, flag stored),
 * 6 slab sums of the draw done, 7 draw done, 8 arrival counted on the row,
 * 9 unit finished, 16+w warp w's share of the statistics pass done (w < 16).  Slots a unit does not reach keep what the caller put there.  stamps = NULL
 * switches it off.  The buffer (dev, 16*units*SPECDEC_STAMP_SLOTS bytes) stays the caller's.
 */
#define SPECDEC_STAMP_SLOTS 32
int specdec_set_phase_stamps(specdec_ctx* ctx, uint64_t* stamps, size_t units);

/*
 * Verify and correct one speculation round for B independent rows
 * (Algorithm 2; Algorithm 1 after its drafting loop; rejection step of Appendix C).
 *
 *   target_logits dev [B, K+1, V]  logits of the target model; row i scores position i,
 *                                  row cand_len[b] is the "p_{K+1}" row of sequence b
 *   draft_logits  dev [B, K, V]    logits of the draft model
 *   dtype                          element type of both logit tensors
 *   cand_tokens   dev [B, K] int32 drafted tokens y_i; entries at i >= cand_len[b] ignored
 *   cand_len      dev [B] int32    candidates per row, 0 <= L <= K; NULL means L = K
 *   uniforms      dev [B, K+1] f32 [b,i<K] = r_i of the accept test, [b,K] = the uniform
 *                                  that draws y' (one fixed slot whatever cand_len[b] is)
 *   temperature                    both models' logits are divided by it; must be > 0
 *   n_accepted    dev out [B] int32  n = min({i < L : r_i >= p_i(y_i)/q_i(y_i)} U {L})
 *   next_token    dev out [B] int32  y': inverse-CDF draw (vocabulary order, smallest j with
 *                                  sum_{v<=j} w_v > u * sum_v w_v) from w = (p_n - q_n)_+ if
 *                                  n < L, from w = p_L otherwise
 *   accept_ratio  dev out [B, K] f32 or NULL: min(1, p_i(y_i)/q_i(y_i)) for i < L, 0 beyond
 *   row_stats     dev out [B, K+1, 4] f32 (16-byte aligned) or NULL:
 *                                  {lse_p, lse_q, p_i(y_i), q_i(y_i)} with
 *                                  lse = log sum_v exp(logit_v / T); the bonus position L
 *                                  holds {lse_p, 0, 0, 0}; positions > L hold zeros
 *   resid_mass    dev out [B] f32 or NULL: sum_v (p_n - q_n)_+ at the first rejection,
 *                                  1 when every candidate was accepted
 *   flags                          SPECDEC_VERIFY_* kernel selection (0 = automatic), optionally | SPECDEC_VERIFY_EARLY_EXIT
 *
 * Logit rows at positions the method does not need (i > cand_len[b] of the target,
 * i >= cand_len[b] of the draft) are never read.  Arithmetic is fp32 (exponentials by
 * ex2.approx), the inverse-CDF prefix above 256-element slabs is accumulated in fp64.
 * Errors: EINVAL (null pointer, B/K/V < 1, temperature <= 0 or not finite, unknown
 * dtype/flags), EUNSUPPORTED (B or K beyond the context, V > 2^22, STREAM kernel
 * requested for rows that are not 16-byte aligned), ECUDA.
 */
int specdec_verify_correct(specdec_ctx* ctx,
                           const void* target_logits, const void* draft_logits, specdec_dtype dtype,
                           const int32_t* cand_tokens, const int32_t* cand_len,
                           const float* uniforms, float temperature,
                           int B, int K, int V,
                           int32_t* n_accepted, int32_t* next_token,
                           float* accept_ratio, float* row_stats, float* resid_mass,
                           uint32_t flags, void* stream);

/*
 * Verify and correct under top-k sampling (Appendix D.1: the paper decodes with top-k sampling,
 * k = 50).  In every row of both models the logits below the row's k-th largest value count as
 * -inf (ties with the k-th largest are kept); Algorithm 2 then runs on the filtered distributions
 * exactly as in specdec_verify_correct.  A drafted token outside the target's kept set is rejected
 * with certainty; y' always lies in the target's kept set.  top_k >= V is the unfiltered
 * operation.  Arguments as for specdec_verify_correct; 1 <= top_k <= 256 (or >= V).
 * The kept logits are evaluated like the unfiltered ones (fp32 terms, fp64 prefix sums).  Logits equal to the k-th largest are all
 * kept.  Where more than 2048 logits of a target row, or 4096 of a draft row, are kept that way the
 * call sets SPECDEC_DATA_TOPK_TIES: an accept test it touches reports n_accepted = -1, a draw it
 * touches next_token = -1.
 */
int specdec_verify_correct_topk(specdec_ctx* ctx,
                                const void* target_logits, const void* draft_logits, specdec_dtype dtype,
                                const int32_t* cand_tokens, const int32_t* cand_len,
                                const float* uniforms, float temperature, int top_k,
                                int B, int K, int V,
                                int32_t* n_accepted, int32_t* next_token,
                                float* accept_ratio, float* resid_mass, void* stream);

/*
 * Greedy verification (Section 4.1: the deterministic setting in which both models decode
 * greedily).  The drafted tokens are given; candidate i is kept while it equals the target's
 * argmax at position i, the first mismatch is replaced by that argmax, and when all cand_len[b]
 * candidates match, the target's argmax at position cand_len[b] is appended.  Only target rows
 * 0..cand_len[b] are read.  Ties in a row resolve to the lowest token index.
 *
 *   target_logits dev [B, K+1, V], cand_tokens dev [B, K] int32, cand_len dev [B] int32 or NULL
 *   n_accepted    dev out [B] int32   number of leading candidates equal to the target's argmax
 *   next_token    dev out [B] int32   target argmax at position n_accepted[b]
 *   target_argmax dev out [B, K+1] int32 or NULL: argmax of every row that was read, -1 elsewhere
 * Errors and device-side data checks as for specdec_verify_correct.
 */
int specdec_verify_greedy(specdec_ctx* ctx, const void* target_logits, specdec_dtype dtype,
                          const int32_t* cand_tokens, const int32_t* cand_len,
                          int B, int K, int V,
                          int32_t* n_accepted, int32_t* next_token, int32_t* target_argmax,
                          void* stream);

/*
 * Sampling one token per row from softmax(logits / temperature): the drafting step y_i ~ q_i of
 * Algorithm 1 and, on the target's logits, the K = 0 case of Algorithm 2 (a round with no candidates
 * draws y' ~ p_1).  The draw is the inverse CDF in vocabulary order at uniforms[b], the rule
 * specdec_verify_correct uses for y', so a drafted token and a verification of it share one
 * definition of "sample".  With 1 <= top_k <= 256 the row is first restricted to its top_k largest
 * logits (ties with the k-th kept); top_k <= 0 or >= V samples from the whole vocabulary.
 *
 *   logits   dev [B, V] row-major, dtype;  uniforms dev [B] fp32 in [0,1);  tokens dev out [B] int32
 * Errors as for specdec_verify_correct (B <= max_B).
 */
int specdec_sample(specdec_ctx* ctx, const void* logits, specdec_dtype dtype, const float* uniforms,
                   float temperature, int top_k, int B, int V, int32_t* tokens, void* stream);

/*
 * Verify/correct on logits split along the vocabulary (what a tensor-parallel output layer
 * produces; the paper shards its 70B target over several GPUs, Appendix D.1).  Rank r of n_shards
 * holds columns [v_offset, v_offset + V_shard) of both models' logits for all B rows.  Algorithm 2
 * then needs two small exchanges, which the CALLER performs between three local calls (any
 * all-gather will do; nothing here touches another GPU's memory or waits for another rank):
 *
 *   1. specdec_shard_stats   -> stats [B, K+1, 8] fp32 per rank; all-gather -> stats_all [n_shards, B, K+1, 8]
 *   2. specdec_shard_accept  -> n_accepted (identical on every rank), row_norm, and this rank's
 *                               mass [B] fp64 of the weights y' is drawn from; all-gather -> mass_all [n_shards, B]
 *   3. specdec_shard_draw    -> next_token[b] on the one rank whose columns contain the draw, -1 on
 *                               the others; a max-reduction over ranks yields next_token.
 *
 * The results equal specdec_verify_correct on the concatenated logits up to fp32 summation order.
 * cand_tokens hold global token ids; V is the whole vocabulary (range check).  A drafted token that
 * no rank, or more than one, holds marks the row bad (n_accepted = next_token = -1).
 * n_shards <= SPECDEC_SHARD_MAX_RANKS.  All pointers are device memory; mass / mass_all are fp64.
 */
#define SPECDEC_SHARD_STATS_WIDTH 8
#define SPECDEC_SHARD_MAX_RANKS 64
typedef struct specdec_shard {
    const void* target_logits;  /* dev [B, K+1, V_shard] row-major */
    const void* draft_logits;   /* dev [B, K,   V_shard]           */
    specdec_dtype dtype;
    int V_shard;                /* columns held by this rank        */
    int v_offset;               /* global token id of local column 0 */
    int V;                      /* size of the whole vocabulary     */
} specdec_shard;

int specdec_shard_stats(specdec_ctx* ctx, const specdec_shard* shard,
                        const int32_t* cand_tokens, const int32_t* cand_len, float temperature,
                        int B, int K, float* stats, void* stream);
int specdec_shard_accept(specdec_ctx* ctx, const specdec_shard* shard,
                         const float* stats_all, int n_shards,
                         const int32_t* cand_len, const float* uniforms, float temperature,
                         int B, int K,
                         int32_t* n_accepted,   /* dev out [B]                                  */
                         float* accept_ratio,   /* dev out [B, K] or NULL                       */
                         float* row_norm,       /* dev out [B, 4], 16-byte aligned: input of _draw */
                         double* mass,          /* dev out [B]                                  */
                         void* stream);
int specdec_shard_draw(specdec_ctx* ctx, const specdec_shard* shard,
                       const float* stats_all, const double* mass_all, int n_shards, int rank,
                       const int32_t* n_accepted, const int32_t* cand_len, const float* uniforms,
                       const float* row_norm, float temperature, int B, int K,
                       int32_t* next_token,     /* dev out [B]: -1 unless this rank draws the row */
                       float* resid_mass,       /* dev out [B] or NULL                            */
                       void* stream);

/*
 * Same operation with HOST input and output buffers: copies the inputs to device staging
 * buffers owned by the context (allocated or grown on first use), runs the kernels, copies
 * n_accepted / next_token (and accept_ratio when not NULL) back and synchronises `stream`
 * before returning.  Pinned host memory lets the copies run at full PCIe rate.
 */
int specdec_verify_correct_host(specdec_ctx* ctx,
                                const void* target_logits, const void* draft_logits, specdec_dtype dtype,
                                const int32_t* cand_tokens, const int32_t* cand_len,
                                const float* uniforms, float temperature,
                                int B, int K, int V,
                                int32_t* n_accepted, int32_t* next_token, float* accept_ratio,
                                uint32_t flags, void* stream);

/*
 * Acceptance-prediction head (Eq. 3; architecture of Section 5.1):
 *   x_0 = hidden;  x_k = x_{k-1} + SiLU(W_k x_{k-1} + b_k), k = 1..depth;
 *   accept_prob = sigmoid(w_out . x_depth + b_out).
 * All tensors bf16 on the device; W_k is [d, d] stored (out, in) like a linear layer's
 * weight; b_k [d] may be NULL (zero).  GEMMs run on tcgen05 tensor cores with fp32
 * accumulation; activations between blocks are rounded to bf16.
 */
typedef struct {
    const void* const* W;   /* host array of `depth` dev pointers, each bf16 [d, d]        */
    const void* const* b;   /* host array of `depth` dev pointers (bf16 [d]) or NULL entries; may be NULL */
    const void* w_out;      /* dev bf16 [d]                                                */
    float b_out;
    int d;                  /* hidden width, multiple of 128                               */
    int depth;              /* number of residual blocks D, 0 <= D <= 8                    */
} specdec_head;

/*
 *   hidden      dev [B, K, d] bf16   final hidden state e_i of each drafted token
 *   accept_prob dev out [B, K] f32   sigmoid(f_theta(e_i))
 * Errors: EINVAL, EUNSUPPORTED (d not a multiple of 128, B*K or d beyond the context), ECUDA.
 */
int specdec_accept_head(specdec_ctx* ctx, const void* hidden, const specdec_head* head,
                        int B, int K, float* accept_prob, void* stream);

/*
 * Threshold stop rule (Section 4.3; loop of Algorithm 1): for each row the first 0-based
 * position j with 1 - prod_{i<=j} accept_prob[b,i] > h (strict), scanning i < cand_len[b]
 * (K when cand_len is NULL).  stop_pos[b] = j, or cand_len[b] (resp. K) if the rule never
 * fires.  Products are formed sequentially in fp32.  A cand_len[b] outside [0, K] gives
 * stop_pos[b] = -1 and sets SPECDEC_DATA_BAD_LENGTH in the device status word; the row is not read.
 *   accept_prob dev [B, K] f32, cand_len dev [B] int32 or NULL, stop_pos dev out [B] int32
 */
int specdec_stop(specdec_ctx* ctx, const float* accept_prob, const int32_t* cand_len,
                 float h, int B, int K, int32_t* stop_pos, void* stream);

/*
 * One trip of Algorithm 1's drafting loop for B sequences (the online form of specdec_stop):
 *   p_hat[b] <- p_hat[b] * accept_prob_step[b];   stop[b] = (1 - p_hat[b] > h) ? 1 : 0.
 * The caller starts a speculation round with p_hat = 1 and calls this after each drafted token
 * with the head's output for that token (specdec_accept_head with K = 1).
 *   accept_prob_step dev [B] f32, p_hat dev in/out [B] f32, stop dev out [B] int32
 */
int specdec_stop_step(specdec_ctx* ctx, const float* accept_prob_step, float* p_hat, float h, int B,
                      int32_t* stop, void* stream);

/*
 * Self-test of the kernels' failure handling (no counterpart in the paper).  Every in-kernel wait
 * of this library is bounded: when it runs out the kernel sets SPECDEC_DATA_WAIT_LIMIT in the
 * status word and carries on instead of hanging.  This call launches a one-thread kernel that
 * waits, with a budget of 4096 polls, on a barrier nothing will ever complete; afterwards
 * specdec_device_status() must report SPECDEC_DATA_WAIT_LIMIT and the context must still work.
 */
int specdec_selftest_wait_limit(specdec_ctx* ctx, void* stream);

/*
 * Allocation-free variant of specdec_verify_correct.  The paper has no counterpart: this entry
 * point exists for callers that cannot call cudaMalloc -- a serving process that has given all
 * device memory to its own pool, a plugin whose host forbids allocations after start-up, a
 * latency-critical loop that cannot afford an allocation's implicit synchronisation.  It needs
 * no context (creating one allocates).  Its scratch is one fixed array of about 256 KB inside
 * the library's device image, present on every GPU that loads the library until the process ends.
 *
 * Inputs and outputs are as for specdec_verify_correct (all "dev", on the CURRENT device),
 * without the optional probability outputs.  data_status (dev, may be NULL) is a word the caller
 * has zeroed; SPECDEC_DATA_* bits are OR-ed into it when a token or length is out of range.
 * err/err_len: host buffer that receives a message when the return value is not SPECDEC_OK
 * (may be NULL/0).
 *
 * Limits: B * (K+1) <= SPECDEC_STATIC_MAX_UNITS and V <= SPECDEC_STATIC_MAX_V; larger problems
 * return SPECDEC_EUNSUPPORTED with a message and launch nothing.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, no
 * allocation); make that first call outside any stream capture.  Every call on a device shares
 * the one array, which keeps the previous call's contents: the library clears what must start
 * from zero on `stream` before the kernel, so calls on one stream are safe back to back, but two
 * calls whose GPU work overlaps (different streams, different host threads) race on it and give
 * wrong results.  Calls no cudaMalloc, cudaFree or any other allocating routine.
 */
#define SPECDEC_STATIC_MAX_UNITS 16384
#define SPECDEC_STATIC_MAX_V     262144
int specdec_verify_correct_static(const void* target_logits, const void* draft_logits, specdec_dtype dtype,
                                  const int32_t* cand_tokens, const int32_t* cand_len,
                                  const float* uniforms, float temperature,
                                  int B, int K, int V,
                                  int32_t* n_accepted, int32_t* next_token,
                                  uint32_t* data_status, void* stream, char* err, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* SPECDEC_H_ */
