/*
 * pc.h -- C ABI of the Pilot-Commit group-rollout engine for NVIDIA B200 (sm_100a).
 *
 * The library generates the rollouts of group-based RL post-training the way the
 * Pilot-Commit method spends them (Section 3.3 of the paper): every prompt of a
 * sampling batch is evaluated once, its key/value cache stays resident and is
 * shared by all rollouts of its group in both the pilot stage (n_pilot rollouts per
 * prompt) and the commit stage (n_commit more rollouts for the prompts that pass the
 * pilot filter); rewards of each group are reduced to the statistics of Eq. 3, the
 * pilot filter / eviction / commit allocation of Algorithm 1 is evaluated on the
 * device, and the group-relative advantages of Section 3.1 are produced for the
 * union of pilot and commit rollouts.
 *
 * Conventions
 *  - Every function returns an int status (PC_OK = 0).  Errors found on the host
 *    (bad arguments, shapes, alignment, capacity) are returned before anything is
 *    launched.  Nothing here synchronises the stream: work is asynchronous.
 *  - The caller owns all device memory: weights, KV arenas, workspace, inputs,
 *    outputs.  The library calls no device allocator.  Two entry points use driver
 *    resources of their own, stated there: pc_set_workspace copies small tables into
 *    the workspace with a synchronous cudaMemcpy, and pc_decode_run creates one CUDA
 *    stream per context and instantiates CUDA graphs (which the driver backs with
 *    memory of its own); both are released by pc_destroy.
 *  - "device" / "host" in a comment says where a pointer must point.
 *  - Matrices are row-major [out_features, in_features] in the model's storage type
 *    (dtype): float (PC_DTYPE_F32) or bfloat16 (PC_DTYPE_BF16).  Norm gains and
 *    biases are always float arrays.  The residual stream, softmax, logits and all
 *    statistics are float; dot products accumulate in float.
 *  - KV arena layout (prompt arena and suffix arena alike):
 *        [n_layers][2 (0 = K after RoPE, 1 = V)][n_kv_heads][n_slots][head_dim]
 *    in the model's storage type (bf16 models: K and V planes IEEE half, still
 *    2 bytes per element); a "slot" holds one token position.  A prompt or a
 *    rollout owns a contiguous range of slots given by its first slot (int64).
 *  - Index arrays are int32, slot numbers and token-buffer indices int64.
 *  - Device-side anomalies set *dev_error_flag (see pc_set_workspace) to a non-zero
 *    code and skip the access; no kernel traps.  What is checked: KV slot ranges
 *    against their arenas, token ids against the vocabulary, every bounded wait, and
 *    -- once the caller has stated the sizes with pc_set_index_bounds -- row_prompt
 *    against the per-prompt arrays and row_tok_index against the token buffer (a row
 *    that fails is switched off for the step).  Other index arrays (row_kv_start,
 *    group_row_start, logits_row, out_index of pc_sample) are the caller's
 *    responsibility.
 */
#ifndef PC_H_
#define PC_H_

#include <stddef.h>
#include <stdint.h>

#if defined(PC_BUILDING_LIB) && defined(__GNUC__)
#define PC_API __attribute__((visibility("default")))
#else
#define PC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PC_OK = 0,
    PC_ERR_INVALID_ARG = 1,   /* null pointer, negative count, bad enum                      */
    PC_ERR_SHAPE = 2,         /* model dimensions the kernels do not support                 */
    PC_ERR_ALIGNMENT = 3,     /* a pointer is not aligned to 16 bytes (256 for the workspace) */
    PC_ERR_CAPACITY = 4,      /* more rows / tokens than the workspace was sized for         */
    PC_ERR_UNSUPPORTED = 5,
    PC_ERR_CUDA = 6,          /* a CUDA runtime / driver call failed; see pc_last_cuda_error */
    PC_ERR_NO_WORKSPACE = 7
};

enum { PC_DTYPE_F32 = 0, PC_DTYPE_BF16 = 1 };

/* Status of a prompt after the pilot stage (Section 3.3; Algorithm 1, Filter / Commit). */
enum {
    PC_STATUS_COMMIT = 0,      /* passed the filter and received n_commit more rollouts          */
    PC_STATUS_BUFFERED = 1,    /* passed the filter but b_t prompts were already selected         */
    PC_STATUS_DEFER_HARD = 2,  /* p_hat < p_lower                                                */
    PC_STATUS_SKIP_EASY = 3,   /* p_hat > p_upper                                                */
    PC_STATUS_LOW_VARIANCE = 4 /* pc_allocate_variance: pilot reward variance below the threshold */
};

typedef struct pc_ctx pc_ctx;

/* Qwen2/3-style pre-norm decoder (the model families of Section 4.1). */
typedef struct pc_model_desc {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    float rms_eps;
    float rope_theta;
    int32_t dtype;       /* PC_DTYPE_*: type of matrices, embedding and KV arenas          */
    int32_t tied_embed;  /* 1: the LM head is the embedding matrix                         */
    int32_t qk_norm;     /* 1: per-head RMSNorm of q and k over head_dim, before RoPE      */
    int32_t qkv_bias;    /* 1: q/k/v projections have a bias                               */
    int32_t half_gemm;   /* bf16 models only.  1: every matrix that feeds a GEMM (wqkv, wo, w_gate_up,
                          * w_down, lm_head) is IEEE half (binary16) instead of bfloat16 and the
                          * activation operands of those GEMMs are rounded to half: three more
                          * mantissa bits at the same bytes and flops, which takes the place of the
                          * second bf16 operand (value + rounding remainder) the bfloat16 path needs
                          * for QKV, output projection and LM head.  lm_head must then be given even
                          * when tied_embed = 1 (a half copy of the embedding, which itself stays
                          * bfloat16 for the token lookup).  A bfloat16 weight converts to half exactly
                          * unless it is below 2^-14 in magnitude (then to within 2^-25).  Activations
                          * and V values that do not fit half (|x| > 65504, or NaN) are stored saturated
                          * and reported as code 5 in *dev_error_flag.                                    */
} pc_model_desc;

/* Device pointers to the weights.  The per-layer members are HOST arrays of n_layers
 * DEVICE pointers; the arrays are copied by pc_create, the tensors are not.
 *   embed      [vocab, d_model]                      lm_head [vocab, d_model] or NULL if tied
 *   final_norm [d_model] float
 *   attn_norm  [d_model] float                       mlp_norm [d_model] float
 *   wqkv       [(Hq + 2 Hkv) * head_dim, d_model]    rows: all q heads, then k heads, then v heads
 *   bqkv       [(Hq + 2 Hkv) * head_dim] float, or NULL array when qkv_bias = 0
 *   q_norm, k_norm [head_dim] float, or NULL arrays when qk_norm = 0
 *   wo         [d_model, Hq * head_dim]
 *   w_gate_up  [2 * d_ff, d_model]   INTERLEAVED: row 2j = gate row j, row 2j+1 = up row j
 *   w_down     [d_model, d_ff]
 *   With half_gemm = 1 wqkv, wo, w_gate_up, w_down and lm_head are IEEE half; embed stays bfloat16.
 */
typedef struct pc_weights {
    const void* embed;
    const void* lm_head;
    const float* final_norm;
    const float* const* attn_norm;
    const void* const* wqkv;
    const float* const* bqkv;
    const float* const* q_norm;
    const float* const* k_norm;
    const void* const* wo;
    const float* const* mlp_norm;
    const void* const* w_gate_up;
    const void* const* w_down;
} pc_weights;

/* Seeded sampling (Section 4.2: temperature 1.0, top_p 1.0 in training). */
typedef struct pc_sample_params {
    float temperature;   /* > 0 */
    uint64_t seed;
} pc_sample_params;

/* Pilot filter, eviction and commit allocation (Section 3.3, 3.4; defaults of Section 4.2:
 * p_lower 0.125, p_upper 0.75, p_solve 1.0). */
typedef struct pc_alloc_params {
    double p_lower, p_upper, p_solve;
    int32_t n_commit;   /* rollouts added to a committed prompt */
    int32_t b_t;        /* at most this many prompts commit     */
} pc_alloc_params;

PC_API const char* pc_status_string(int status);
/* Text of the last CUDA error seen by this thread inside the library (host pointer, static storage). */
PC_API const char* pc_last_cuda_error(void);

/* Number of kernels this library has launched since it was loaded (host counter, all contexts and
 * host threads; updated atomically). */
PC_API uint64_t pc_launch_count(void);
/* Number of decode steps this context has captured and instantiated as CUDA graphs so far (see pc_decode_run). */
PC_API uint64_t pc_capture_count(const pc_ctx* ctx);

/* Builds a context: copies the description and the pointer tables (host memory only)
 * and, for bf16 models, encodes the TMA descriptors of the weight matrices.  Needs a
 * current CUDA device for bf16 models.  Shapes: head_dim in {64, 128}; n_q_heads a
 * multiple of n_kv_heads with ratio <= 8; d_model, d_ff, q/kv widths multiples of 8;
 * bf16 additionally needs d_model, d_ff and Hq*head_dim multiples of 64. */
PC_API int pc_create(const pc_model_desc* desc, const pc_weights* weights, pc_ctx** out);
PC_API void pc_destroy(pc_ctx* ctx);

/* Scratch the kernels need for at most max_rows concurrent rollouts per decode step and
 * max_prefill_tokens packed prompt tokens per prefill call. */
PC_API int pc_workspace_bytes(const pc_ctx* ctx, int max_rows, int max_prefill_tokens, size_t* out_bytes);
/* dev_ws: device, 256-byte aligned, at least `bytes` long, untouched by the caller while
 * work of this context is in flight.  dev_error_flag: device int32, zeroed by the caller;
 * kernels store a non-zero code there when they meet an out-of-range index. */
PC_API int pc_set_workspace(pc_ctx* ctx, void* dev_ws, size_t bytes, int max_rows, int max_prefill_tokens,
                     int32_t* dev_error_flag);

/* Tuning aid: forces the tile width (64 or 256 output columns) and the number of K-slices of the bf16 tensor-core
 * GEMMs instead of the built-in choice.  spec (host string) is a comma-separated list of name=WIDTHxSLICES with name
 * in {qkv, o, gu, dn, lm} (QKV, output, gate/up, down projection, LM head), e.g. "dn=256x4,o=64x2"; names left out,
 * NULL or "" keep the built-in choice.  The slice count is clamped to what the workspace holds for the step's row
 * bound; gate/up and the LM head never split.  Where the QKV and output projections run with the fused epilogues
 * (pc_set_fused_epilogues) only the width applies to them: 128 or 256 for QKV (whole heads per tile; 128 is accepted for
 * this case only and otherwise read as 64), 64 or 256 for the output projection.  Results stay deterministic for a
 * fixed plan.  Drops captured decode steps.  The paper has no counterpart. */
PC_API int pc_set_gemm_plan(pc_ctx* ctx, const char* spec);

/* Self-test of the bounded waits every kernel here uses on its mbarriers: launches one warp that waits, for at most
 * spin_limit polls (1 .. 2^20), on a barrier nothing arrives at; the wait gives up, stores DEV_ERR_WAIT_TIMEOUT (3) in
 * *dev_error_flag (device int32) and the kernel returns normally, so the context stays usable.  No counterpart in the paper. */
PC_API int pc_selftest_wait_timeout(void* stream, uint32_t spin_limit, int32_t* dev_error_flag);

/* Sizes of the caller's per-prompt arrays (prompt_len, prompt_kv_start, prompt keys) and of the token buffer, so that
 * the decode steps can check row_prompt and row_tok_index against them (see "Device-side anomalies" above).  0 = not
 * stated, not checked (the default). */
PC_API int pc_set_index_bounds(pc_ctx* ctx, int n_prompts, int64_t n_tokens);

/* bf16 models with half_gemm = 1 and head_dim 128, passes of more than 256 rows.  1 (the default): two row-wise kernels
 * of every layer run inside GEMM epilogues instead -- bias / QK-norm / RoPE / KV append in the QKV projection's, and the residual add, the operand of the
 * gate/up projection and the RMSNorm's sum of squares in the output projection's, the norm's 1/rms being applied by the
 * gate/up epilogue (RMSNorm(h; g) W^T = rstd * ((h * g) W^T)).  The two projections then run without K split, which is why
 * smaller passes keep the separate kernels (their projections need the split to fill the GPU).  0: one kernel per
 * operation throughout, as for every other model type.  A value n > 1: the fused form from passes of n rows on (a
 * measurement aid: below 257 rows it is slower).  Same mathematics, different rounding order (both inside the
 * tolerances the tests state).  Drops captured decode steps.  The paper has no counterpart. */
PC_API int pc_set_fused_epilogues(pc_ctx* ctx, int on);

/* bf16 models.  mask: one bit per kernel (1 QKV, 2 output, 4 gate/up, 8 down projection, 16 LM head, 32 shared-prefix
 * attention of decode steps), 0 .. 63; the default is 63.  A kernel whose bit is set is launched as a programmatic
 * dependent of the kernel before it (a row norm, the QKV post-processing, the attention merge or a projection, all of
 * which signal their dependents as soon as they start).  A projection's CTAs set up their barriers and tensor memory
 * and request their first weight tiles while that kernel is still running; the attention kernel requests its first
 * prompt K/V tiles (written by an earlier call).  Both wait for the kernel before them (griddepcontrol.wait) before they
 * touch activations or any output.  Results are bit-identical to mask 0 (plain stream order); only the start of each
 * kernel moves.  Projections of passes of 129 .. 256 rows (two row tiles: measured slower with it) and steps that record
 * phase events (pc_profile_step) run in plain stream order whatever the mask.  Drops captured decode steps.  The paper
 * has no counterpart. */
PC_API int pc_set_dependent_launch(pc_ctx* ctx, int mask);

/* bf16 models, decode steps that only sample (no logits_out, no log-probability buffer): 1 draws the token in
 * the epilogue of the LM-head GEMM -- per half tile of the vocabulary the largest and second-largest perturbed score
 * and the arg-max, folded per row by a small second kernel -- so the step's [rows, vocab] logits are never written or read
 * back; 0 (the default) stores the logits and runs the stand-alone sampler on them.  Both draw exactly the same tokens
 * (Section 4.2: T = 1.0, top_p = 1.0; pc_sample states the rule): the tiles of a row share a running lower bound of the
 * row's second-best score, so which candidates a tile scores depends on timing, the folded result does not.  The
 * epilogue form is not the faster one on B200 (LM head + draw at 2048 rows: 2.37 ms against 0.90 + 0.60 ms; at 64 rows
 * 0.17 against 0.15 ms): the Philox arithmetic needs many warps per scheduler to reach the integer pipes' rate, and a
 * GEMM CTA has room for eight epilogue warps.  It is kept for callers that cannot afford the [rows, vocab] logits
 * buffer.  Drops captured steps. */
PC_API int pc_set_fused_sampler(pc_ctx* ctx, int on);

/* bf16 models, decode steps: 1 issues the shared-prefix attention kernel and the per-rollout suffix attention
 * kernel of a layer on two streams (the second one is created by the context on first use and released by pc_destroy), so
 * that they can overlap; 0 (the default: measured no faster, both kernels fill the SMs) issues them one after the other.
 * Results are identical.  Drops captured decode steps. */
PC_API int pc_set_attention_overlap(pc_ctx* ctx, int on);

/* How the decode steps of a bf16 model with half_gemm = 1 are issued.  mode 1: everything between two
 * attention calls of a step -- output projection, residual + RMSNorm, gate/up + SwiGLU, down projection, residual +
 * RMSNorm, QKV projection of the next layer and its bias / QK-norm / RoPE / KV append; embedding before the first
 * layer, LM head after the last -- runs as phases of ONE persistent cooperative kernel with grid-wide barriers, the
 * weight tiles of the next GEMM being requested across the barriers.  mode 0 (the default): one kernel per operation.  Both modes
 * run the same arithmetic in the same order and give identical results; models of other types always use mode 0.
 * Drops captured decode steps.  The paper has no counterpart. */
PC_API int pc_set_decode_mode(pc_ctx* ctx, int mode);

/* Tracing aid for mode 1: with a buffer set (device int64, at least pc_chain_trace_words(ctx) words, zeroed by the
 * caller), the first four CTAs of every launch of the persistent kernel store SM clock stamps of their roles per phase:
 * trace[segment + 1][phase][cta][16], events 0..11 = workers begin / barrier passed / done, producer begin / barrier
 * passed / done, first operand tile arrived / MMAs issued, first accumulator ready / epilogues done, kernel begin / end
 * (the last two in phase 0).  NULL switches it off (the default).  Drops captured decode steps.  No counterpart in the paper. */
PC_API int pc_set_chain_trace(pc_ctx* ctx, int64_t* trace, size_t n_words);
PC_API size_t pc_chain_trace_words(const pc_ctx* ctx);

/* Measurement aid: the next pc_decode_step of this context (issued outside any capture, one kernel per operation)
 * records the PC_PROFILE_MARKS CUDA events (cudaEvent_t with timing, created by the caller; NULL entries are skipped) at
 * the boundaries of the operations of decoder layer `layer` and of the step's tail, in stream order:
 *   LAYER_BEGIN | attention RMSNorm | NORM_ATTN | QKV GEMM | QKV | bias / QK-norm / RoPE / KV append | POST |
 *   shared-prefix attention | GROUP | per-rollout suffix attention | SUFFIX | merge | MERGE | output projection | O |
 *   MLP RMSNorm | NORM_MLP | gate/up GEMM + SwiGLU | GATE_UP | down projection | DOWN   ... (other layers) ...
 *   LM_BEGIN | final RMSNorm + LM head | LM_HEAD | sampler | SAMPLE
 * so the time of an operation is the elapsed time between the marks around it.  One-shot; the caller synchronises
 * and reads the times.  float32 models run one attention kernel: GROUP is recorded before it, SUFFIX and MERGE after
 * it.  The paper has no counterpart. */
enum {
    PC_MARK_LAYER_BEGIN = 0, PC_MARK_NORM_ATTN, PC_MARK_QKV, PC_MARK_POST, PC_MARK_GROUP, PC_MARK_SUFFIX, PC_MARK_MERGE, PC_MARK_O,
    PC_MARK_NORM_MLP, PC_MARK_GATE_UP, PC_MARK_DOWN, PC_MARK_LM_BEGIN, PC_MARK_LM_HEAD, PC_MARK_SAMPLE, PC_PROFILE_MARKS
};
PC_API int pc_profile_step(pc_ctx* ctx, int layer, void* const* events, int n_events);

/* Shared prefill (Section 3.1: o ~ pi_theta(. | q); Section 3.3: pilot and commit rollouts of a
 * prompt are drawn from the same pi_theta(. | q), so q is evaluated once).
 * Full causal forward over every prompt of the batch; writes K (after RoPE) and V of every
 * prompt position and layer into the prompt arena and the logits at each prompt's last
 * position.
 *   prompt_tokens   device [total_tokens] int32, prompts packed back to back
 *   prompt_offsets  device [n_prompts + 1] int32, prompt p = tokens[offsets[p] : offsets[p+1]]
 *   total_tokens, max_prompt_len   host scalars describing the same arrays
 *   prompt_kv       device, arena with prompt_slots slots
 *   prompt_kv_start device [n_prompts] int64, first slot of each prompt
 *   last_logits     device [n_prompts, vocab] float, written */
PC_API int pc_prefill_shared(pc_ctx* ctx, void* stream, int n_prompts, const int32_t* prompt_tokens,
                      const int32_t* prompt_offsets, int total_tokens, int max_prompt_len,
                      void* prompt_kv, int64_t prompt_slots, const int64_t* prompt_kv_start,
                      float* last_logits);

/* One autoregressive step for n_rows live rollouts (Section 3.1: pi_theta(o_t | q, o_<t)).
 * Row r belongs to prompt row_prompt[r], is rollout row_rollout[r] of its group and has
 * row_step[r] suffix tokens cached already.  Its input token is tokens[row_tok_index[r]]; the
 * step appends that token's K/V at suffix slot row_kv_start[r] + row_step[r], attends over the
 * prompt's shared KV (prompt_len[p] slots from prompt_kv_start[p]) followed by the rollout's own
 * row_step[r] + 1 suffix slots, and produces the logits of the next token.
 *   logits_out  device [n_rows, vocab] float or NULL
 *   sample      host or NULL.  When given, the next token is drawn as in pc_sample with
 *               step key row_step[r] + 1 and stored at tokens[row_tok_index[r] + 1].
 * Rows of one prompt must be contiguous; group g covers rows
 * group_row_start[g] .. group_row_start[g+1]-1 (device [n_groups + 1] int32), none longer
 * than max_group_rows (host scalar).  All row_* arrays are device [n_rows]. */
PC_API int pc_decode_step(pc_ctx* ctx, void* stream, int n_rows,
                   const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step,
                   const int64_t* row_kv_start, int32_t* tokens, const int64_t* row_tok_index,
                   int n_groups, const int32_t* group_row_start, int max_group_rows,
                   const int32_t* prompt_len, const void* prompt_kv, int64_t prompt_slots,
                   const int64_t* prompt_kv_start, void* suffix_kv, int64_t suffix_slots,
                   float* logits_out, const pc_sample_params* sample);

/* One decode step of a device-resident schedule (see pc_decode_run). */
typedef struct pc_step_desc {
    int32_t n_rows, n_groups, max_group_rows, reserved;
    int64_t row_offset;     /* the step's rows are entries [row_offset, row_offset + n_rows) of the row_* arrays */
    int64_t group_offset;   /* its groups are entries [group_offset, group_offset + n_groups] of group_row_start */
} pc_step_desc;

/* n_steps consecutive decode steps (each exactly a pc_decode_step with sampling and no logits output) over a
 * schedule that already lives on the device: the row_* arrays and group_row_start hold every step's entries back to
 * back and step s uses the slices named by steps[s].  steps_host and steps_dev are the same n_steps descriptors in
 * host and in device memory.  The kernels of a step are captured once per shape class (rows rounded up to 128, groups
 * to a power of two, largest group to a query-tile boundary; per pair of KV arenas) into a CUDA graph and replayed, so
 * the host issues one launch per step; the caller's arrays and sampling parameters are read through a device-resident
 * argument block, so a new schedule, token buffer or seed needs no new capture.  The first call creates a CUDA stream
 * owned by the context (captures run there) and every capture instantiates a graph; pc_destroy, pc_set_workspace,
 * pc_set_gemm_plan and pc_set_decode_mode release them.  The stream must not be capturing.  Steps with n_rows = 0 are
 * skipped.  All other arguments as in pc_decode_step. */
PC_API int pc_decode_run(pc_ctx* ctx, void* stream, int n_steps, const pc_step_desc* steps_host, const pc_step_desc* steps_dev,
                         const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step,
                         const int64_t* row_kv_start, int32_t* tokens, const int64_t* row_tok_index,
                         const int32_t* group_row_start, const int32_t* prompt_len, const void* prompt_kv,
                         int64_t prompt_slots, const int64_t* prompt_kv_start, void* suffix_kv, int64_t suffix_slots,
                         const pc_sample_params* sample);

/* Seeded draw from softmax(logits / T) by Gumbel-max (Section 4.2: T = 1.0, top_p = 1.0):
 *   token = argmin-index argmax_v ( logits[v] / T + g_v ),   g_v = -ln(-ln u_v),
 *   u_v = ((w_v >> 9) + 0.5) * 2^-23, w_v = word (v & 3) of Philox4x32-10 with
 *   key (seed lo, seed hi) and counter (v >> 2, step, rollout, prompt).
 * Row r reads logits row logits_row[r] (NULL: row r), so all rollouts of a group can draw
 * their first token from their prompt's single prefill row.
 *   out_tokens  device int32; token of row r is stored at out_tokens[out_index[r]] (NULL: [r])
 *   out_top2_gap device [n_rows] float or NULL: largest minus second-largest perturbed score
 *   scratch     device, 16-byte aligned, scratch_bytes long, or NULL.  With few rows the vocabulary of a row is
 *               scored by several blocks that leave 16-byte records here (n_rows * up to 32 records are used
 *               when they fit); without scratch one block scores a whole row.  The result is the same. */
PC_API int pc_sample(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row,
              float temperature, uint64_t seed, const int32_t* row_prompt, const int32_t* row_rollout,
              const int32_t* row_step, int32_t* out_tokens, const int64_t* out_index, float* out_top2_gap,
              void* scratch, size_t scratch_bytes);

/* Behaviour log-probability of drawn tokens, the denominator pi_theta_old(o_t | q, o_<t) of the token importance ratio
 * (Eq. 2):  out = logits[token] / T - log sum_v exp(logits[v] / T).  Row r reads logits row logits_row[r] (NULL: r),
 * its token is tokens[tok_index[r]] (NULL: tokens[r]) and the result goes to out_logprob[out_index[r]] (NULL: [r]).
 * All pointers device. */
PC_API int pc_token_logprob(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row,
                            float temperature, const int32_t* tokens, const int64_t* tok_index, float* out_logprob,
                            const int64_t* out_index);

/* With a buffer set (device float, indexed exactly like the token buffer of pc_decode_step / pc_decode_run), every
 * decode step that samples also stores the behaviour log-probability (Eq. 2) of the token it drew at
 * logprobs[row_tok_index[r] + 1].  NULL switches it off (the default). */
PC_API int pc_set_logprob_buffer(pc_ctx* ctx, float* logprobs);

/* Sampling keys of the prompts.  By default the decode steps key a draw by (seed, row_prompt, rollout, step), i.e. by a
 * prompt's index in the arrays of the call.  When pilot rollouts of one sampling batch and commit rollouts of the
 * previous batch's survivors share one decode batch (Section 3.4, "Binding pilot and commit"), a prompt's index in the
 * combined arrays differs from the one it had when its pilot rollouts were drawn; prompt_key (device int32, one entry per
 * prompt of the call, or NULL for the default) supplies the id to use in the key instead, so that a rollout's tokens do
 * not depend on how batches are bound. */
PC_API int pc_set_prompt_keys(pc_ctx* ctx, const int32_t* prompt_key);

/* pc_sample for callers that cannot provide scratch memory.  The paper has no counterpart: this entry point exists for
 * hosts of this library that must not allocate device memory at the moment they sample -- code running inside a
 * stream-ordered region whose allocator is frozen, a plugin that is handed only its input and output buffers, a
 * process whose memory pool is owned by another framework and already exhausted.  pc_sample needs caller-provided
 * scratch to spread a small batch over the GPU; here the same two-pass sampler keeps its per-range records in an array
 * that is part of the library image (2 MiB per GPU that loads the library, held until the process exits).
 *   - at most 4096 rows per call; more is refused with PC_ERR_CAPACITY (pc_last_cuda_error gives the text).
 *   - the first call on each device looks up the array's device address; make that first call outside any stream
 *     capture, with the device that will run the kernels current.
 *   - all calls on a device share the one array and it keeps the previous call's records.  Nothing needs clearing
 *     (a call overwrites every record it later reads), but two calls that overlap on the GPU -- different streams,
 *     or different host threads without ordering -- race on it: order them.
 *   - no cudaMalloc, cudaFree or other allocating call is made.  Arguments and results exactly as pc_sample's. */
PC_API int pc_sample_static(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row,
                            float temperature, uint64_t seed, const int32_t* row_prompt, const int32_t* row_rollout,
                            const int32_t* row_step, int32_t* out_tokens, const int64_t* out_index, float* out_top2_gap);

/* Binary reward of the synthetic workloads, standing in for the verifier R(q, o) in {0, 1} of
 * Section 3.3: reward[i] = 1 if tokens[last_index[i]] < threshold[i] else 0.  All device. */
PC_API int pc_reward_last_token(void* stream, int n, const int32_t* tokens, const int64_t* last_index,
                         const int32_t* threshold, float* reward);

/* Group statistics (Eq. 3, population form) and the pilot estimate p_hat = n_success / n
 * (Section 3.3).  Group g is rewards[group_start[g] : group_start[g] + group_count[g]].
 * Outputs, device [n_groups]: n, n_success (number of rewards equal to 1), mean, var. */
PC_API int pc_group_stats(void* stream, int n_groups, const float* rewards, const int32_t* group_start,
                   const int32_t* group_count, int32_t* n, int32_t* n_success, float* mean, float* var);

/* Pilot filter, eviction and commit allocation (Section 3.3, 3.4; Algorithm 1: Filter, Evict,
 * Commit).  p_hat = (double) pilot_success / pilot_n; keep iff p_lower <= p_hat <= p_upper;
 * evict iff p_hat >= p_solve (independent of the filter); the first b_t kept prompts in batch
 * order get status COMMIT and extra_rollouts = n_commit, later ones BUFFERED.
 * Outputs device: status, extra_rollouts, evict [n_prompts] int32; n_selected [1] int32;
 * total_rollouts [1] int64 = sum(pilot_n) + n_selected * n_commit (the cost of Section 4.3). */
PC_API int pc_allocate(void* stream, int n_prompts, const int32_t* pilot_success, const int32_t* pilot_n,
                const pc_alloc_params* params, int32_t* status, int32_t* extra_rollouts, int32_t* evict,
                int32_t* n_selected, int64_t* total_rollouts);

/* The pilot filter for rewards that are not binary.  Section 3.3 motivates the filter by reward variance (for binary
 * rewards Var = p (1 - p), so p_hat is its proxy) and states that the method applies to any scalar reward; it gives no
 * formula for that case.  Reading taken here: keep a prompt iff the population variance of its pilot rewards (Eq. 3,
 * the float value pc_group_stats returns, compared in double) is at least var_min; the first b_t kept prompts in batch
 * order get status COMMIT and extra_rollouts = n_commit, later ones BUFFERED, the others PC_STATUS_LOW_VARIANCE.  There
 * is no eviction rule in this mode.  For binary rewards and thresholds symmetric about 1/2 it decides exactly like
 * pc_allocate with var_min = p_lower (1 - p_lower).  Outputs as pc_allocate's (no evict array). */
PC_API int pc_allocate_variance(void* stream, int n_prompts, const float* pilot_var, const int32_t* pilot_n, double var_min,
                                int n_commit, int b_t, int32_t* status, int32_t* extra_rollouts, int32_t* n_selected,
                                int64_t* total_rollouts);

/* Group-relative advantage A_i = (r_i - mu) / sigma (Section 3.1) over group g =
 * rewards[group_start[g] : +group_count[g]]; 0 when all rewards of the group are equal, and
 * for groups whose status (device [n_groups] or NULL) is not PC_STATUS_COMMIT.
 * adv: device, same indexing as rewards; only elements inside a group are written. */
PC_API int pc_grpo_advantage(void* stream, int n_groups, const float* rewards, const int32_t* group_start,
                      const int32_t* group_count, const int32_t* status, float* adv);

#ifdef __cplusplus
}
#endif
#endif /* PC_H_ */
