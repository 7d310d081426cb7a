/*
 * depcap.h — C ABI of the DepCap block-step library (CUDA, sm_100a).
 *
 * One call of dc_step runs one block-wise denoising step of a masked diffusion LM on one GPU:
 * the bidirectional transformer forward that re-predicts the candidate window over a cached
 * clean context, fused with the per-step signals DepCap decides on, and the block-boundary
 * decision.  dc_select then picks the conflict-free subset of tokens to commit.
 *
 * Paper: "DepCap: Adaptive Block-Wise Parallel Decoding for Efficient Diffusion LM Inference".
 * Passages each call follows are cited at the call.  Notation follows the paper:
 *   B        the last decoded block (length Lb), c the decoded context before it
 *   window   the L_window = min(L_max, L_remain) candidate positions after the frontier
 *   p_curr   p(Z_k | c, b): prediction with the last block decoded      (Section 4.2 / 4.4)
 *   p_prev   p(Z_k | c):    prediction with the last block still masked
 *   I_k      KL(p_curr || p_prev), last-block influence                  (Eq. 3)
 *   H_k      entropy of p_curr                                           (Section 4.2)
 *   S_k      I~_k - lambda * H~_k, dependency score                      (Eq. 4)
 *   c_i      max_v p_i(v), confidence; yhat_i its argmax                 (Section 4.3)
 *   D_ij     log p_i(yhat_j) + log p_j(yhat_i), conflict score           (Eq. 6)
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the GPU that was current in dc_create;
 *     "host" pointers are ordinary host memory read during the call.
 *   - All buffers are owned by the caller.  The library allocates only its own workspace, in
 *     dc_create, and frees it in dc_destroy.  Weight and cache pointers are borrowed: they must
 *     stay valid and unchanged while a call that reads them is in flight.
 *   - dc_step / dc_select / dc_boundary only enqueue work on the context's stream and return;
 *     outputs are valid after the caller synchronises that stream.
 *   - Every call returns a dc_status.  Argument and shape errors are detected on the host before
 *     anything is launched and leave the outputs untouched; dc_last_error gives the reason.
 *     Conditions detected on the device (an expired bounded wait) are written to status[b].
 *   - Calls on one context are not thread-safe.
 *   - Matrix layouts are row-major; weights are [out_features, in_features].
 *   - Element type of weights, caches and h_final_in is dc_config.dtype (fp32 or bf16).  In the
 *     bf16 path every GEMM input is rounded to bf16, accumulation and the residual stream are fp32.
 */
#ifndef DEPCAP_H_
#define DEPCAP_H_

#include <stdint.h>

#if defined(__GNUC__)
#define DC_API __attribute__((visibility("default")))
#else
#define DC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dc_status {
  DC_OK = 0,
  DC_ERR_INVALID_ARG = 1, /* null pointer, bad enum value, negative size                    */
  DC_ERR_SHAPE = 2,       /* a length exceeds the capacity given to dc_create               */
  DC_ERR_UNSUPPORTED = 3, /* a shape the kernels cannot handle (see dc_create)              */
  DC_ERR_NOMEM = 4,       /* workspace allocation failed                                    */
  DC_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed                            */
  DC_ERR_TIMEOUT = 6,     /* device side: a bounded wait inside a kernel ran out            */
  DC_ERR_INDEX = 7,       /* device side: a token id outside [0, vocab)                     */
  DC_ERR_NUMERIC = 8      /* device side: a window position without any finite logit (NaN or  */
                          /* infinite hidden state); its pred_id is reported as mask_id      */
} dc_status;

enum { DC_F32 = 0, DC_BF16 = 1 };                       /* dc_config.dtype             */
enum { DC_NORM_MAX = 0, DC_NORM_MINMAX = 1, DC_NORM_NONE = 2 };   /* dc_config.norm_mode */
enum { DC_BOUNDARY_FIRST_NEG = 0, DC_BOUNDARY_CUMULATIVE = 1 };   /* dc_config.boundary_mode */
enum { DC_CAP_LITERAL = 0, DC_CAP_STRICT = 1 };                   /* dc_config.cap_mode  */
enum { DC_IMPL_AUTO = 0, DC_IMPL_SIMT = 1 };                      /* dc_config.impl      */
enum { DC_MAX_BATCH = 32, DC_MAX_WINDOW = 256 };

/* dc_step_in.flags */
enum {
  DC_STEP_INFLUENCE = 1, /* also run the prev variant and reduce I_k (Eq. 3)                */
  DC_STEP_BOUNDARY = 2,  /* run the boundary rule (Section 4.2) and write block_len         */
  DC_STEP_CARRIED_PREV = 8, /* p_prev comes from rows the caller carried over from an earlier step
                            (h_prev_in, prev_len) instead of a second variant in this pass: the
                            stack runs the curr rows only (half the rows).  This is how the
                            paper's own implementation obtains the two distributions (appendix,
                            Implementation Approximation).  Not together with DC_STEP_INFLUENCE */
  DC_STEP_EXPORT_KV = 4  /* append the last decoded block's K / V (curr variant, every layer) to
                            the caches at keys ctx_len[b] .. ctx_len[b] + last_len[b] - 1: the
                            library WRITES k_cache / v_cache there (block-wise cache reuse,
                            Section 4.1);
                            needs ctx_len[b] + last_len[b] <= max_ctx                        */
};

typedef struct dc_config {
  /* backbone shape (the paper treats the DLM as given; these name it) */
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
  int32_t mask_id;   /* id of [MASK] (Section 3)                                            */
  int32_t dtype;     /* DC_F32 | DC_BF16                                                    */
  float rms_eps;     /* RMSNorm epsilon                                                     */
  float rope_theta;  /* rotary base; pairs (i, i + head_dim/2), angle pos * theta^(-2i/hd)  */
  /* capacities: fix the layouts of caches and outputs */
  int32_t max_batch;  /* <= DC_MAX_BATCH                                                    */
  int32_t max_ctx;    /* multiple of 64                                                     */
  int32_t max_last;   /* longest last decoded block                                         */
  int32_t max_window; /* <= DC_MAX_WINDOW, multiple of 16                                   */
  /* DepCap hyper-parameters ("Hyperparameter settings": 1.2, 8, 128, 0.8, 0.95, -16.0)     */
  float lambda;
  int32_t L_min, L_max;
  float tau_low, tau_high, gamma;
  /* readings of points the paper leaves open */
  int32_t smooth_radius;    /* centered moving average over 2r+1 in-range taps; 0 = off     */
  int32_t norm_mode;        /* how I and H are normalised inside the window                 */
  int32_t boundary_mode;    /* first S_k < 0 (Section 4.2) or first negative running sum    */
                            /* of S_k (the cumulative criterion of Section 4.4)             */
  int32_t cap_mode;         /* Algorithm 1 as printed, or phase 1 also conflict-checked     */
  int32_t forbid_mask_pred; /* 1: [MASK] is removed from the softmax of both variants       */
  int32_t impl;             /* DC_IMPL_AUTO: tensor-core kernels where the shape allows;     */
                            /* DC_IMPL_SIMT: plain CUDA-core kernels only (any shape)       */
  int32_t qkv_bias;         /* 1: the q / k / v projections carry biases (dc_weights.bq/bk/bv), */
                            /* added before the rotation; the Dream backbone (Section 5.1) has */
                            /* them, LLaDA does not.  0: no biases anywhere                    */
} dc_config;

/* Borrowed device pointers.  Per-layer members are HOST arrays of n_layers device pointers. */
typedef struct dc_weights {
  const void* embed;          /* [vocab, d_model]                                           */
  const void* const* wq;      /* [n_q_heads*head_dim, d_model]                              */
  const void* const* wk;      /* [n_kv_heads*head_dim, d_model]                             */
  const void* const* wv;      /* [n_kv_heads*head_dim, d_model]                             */
  const void* const* wo;      /* [d_model, n_q_heads*head_dim]                              */
  const void* const* w_gate;  /* [d_ff, d_model]                                            */
  const void* const* w_up;    /* [d_ff, d_model]                                            */
  const void* const* w_down;  /* [d_model, d_ff]                                            */
  const void* const* norm1;   /* [d_model] gain of the pre-attention RMSNorm                */
  const void* const* norm2;   /* [d_model] gain of the pre-MLP RMSNorm                      */
  const void* final_norm;     /* [d_model]                                                  */
  const void* lm_head;        /* [vocab, d_model] (untied)                                  */
  const void* const* bq;      /* [n_q_heads*head_dim]   biases of the q / k / v projections; */
  const void* const* bk;      /* [n_kv_heads*head_dim]  read only when dc_config.qkv_bias,   */
  const void* const* bv;      /* [n_kv_heads*head_dim]  null otherwise                       */
} dc_weights;

typedef struct dc_step_in {
  int32_t batch; /* sequences in this step, 1..max_batch; sequence b uses cache slot b      */
  int32_t flags; /* DC_STEP_*                                                                */
  /* context cache, device, read-only.  K is stored rotated (post-RoPE).
   *   k_cache [n_layers][max_batch][n_kv_heads][max_ctx][head_dim]
   *   v_cache [n_layers][max_batch][n_kv_heads][head_dim][max_ctx]   (V transposed: keys are
   *           the contiguous axis, which is what the PV product streams)
   * Only the first ctx_len[b] keys of slot b are read; the rest may hold anything.
   * Both may be null when every ctx_len is 0. */
  const void* k_cache;
  const void* v_cache;
  const int32_t* ctx_len;    /* host [batch], 0..max_ctx                                    */
  const int32_t* last_ids;   /* device [batch][max_last]: the last decoded block B          */
  const int32_t* last_len;   /* host [batch], 0..max_last; 0 = no last block (cold start)   */
  const int32_t* win_ids;    /* device [batch][max_window]; mask_id = still masked          */
  const int32_t* win_len;    /* host [batch], 1..max_window: window positions supplied      */
  const int32_t* remain_len; /* host [batch]: L_remain, masked tokens after the frontier    */
  /* Optional, device, [batch][2][max_window][d_model] (curr, prev): replaces the transformer
   * stack's output as the LM-head input (the stack still runs).  For tests and benchmarks that
   * need shaped distributions from random-init weights.  Null in normal use. */
  const void* h_final_in;
  /* DC_STEP_CARRIED_PREV: device [batch][max_window][d_model], model dtype: row k of sequence b is
   * the LM-head input (final-normed hidden state, as h_out of an earlier step gives it) whose
   * distribution serves as p_prev of window position k, for k < prev_len[b] (host [batch],
   * 0..win_len[b]).  Positions k >= prev_len[b] have no earlier prediction: I_k = 0 there, so the
   * boundary rule ends the block at prev_len[b] at the latest; prev_len[b] = 0 is a cold start. */
  const void* h_prev_in;
  const int32_t* prev_len;
  /* Optional, host [batch]: absolute position of the first active row (the frontier).  Null: the
   * rows follow the cached keys, position ctx_len[b] + r.  With a dual cache (the context cache
   * also holds the masked suffix behind the window, Section 5.2) the number of cached keys is no
   * longer the frontier's position: pass it here. */
  const int32_t* pos0;
} dc_step_in;

/* Caller-owned device buffers; rows b >= batch and columns k >= win_len[b] are not written.
 * Any pointer except status may be null to skip that output. */
typedef struct dc_step_out {
  int32_t* pred_id;     /* [batch][max_window] yhat_k                                       */
  float* conf;          /* [batch][max_window] c_k = max_v p_curr(v)                        */
  float* entropy;       /* [batch][max_window] H_k                                          */
  float* influence;     /* [batch][max_window] I_k (0 without a prev variant)               */
  float* lse;           /* [batch][max_window] log-sum-exp of the curr logits               */
  float* xlogp;         /* [batch][max_window][max_window] log p_i(yhat_j)  (Eq. 6 halves)  */
  float* score;         /* [batch][max_window] S_k                (DC_STEP_BOUNDARY)        */
  float* cum_influence; /* [batch][max_window] sum_{j<=k} I_j     (DC_STEP_BOUNDARY)        */
  float* cum_score;     /* [batch][max_window] sum_{j<=k} S_j     (DC_STEP_BOUNDARY)        */
  int32_t* block_len;   /* [batch] next block length L            (DC_STEP_BOUNDARY)        */
  int32_t* status;      /* [batch] DC_OK or a device-side dc_status; required               */
  void* h_out;          /* optional, [batch][max_window][d_model], model dtype: the LM-head input
                           rows of the curr variant, to be carried into a later step's h_prev_in
                           (row k of this window is row k - L of the next one after a block of L) */
} dc_step_out;

typedef struct dc_boundary_in {
  int32_t batch;
  const float* influence;    /* device [batch][max_window]                                  */
  const float* entropy;      /* device [batch][max_window]                                  */
  const int32_t* win_len;    /* host [batch]                                                */
  const int32_t* remain_len; /* host [batch]                                                */
  const int32_t* have_prev;  /* host [batch]; 0 = cold start (L = L_min)                    */
} dc_boundary_in;

typedef struct dc_boundary_out {
  float* score;         /* device [batch][max_window], may be null                          */
  float* cum_influence; /* device [batch][max_window], may be null                          */
  float* cum_score;     /* device [batch][max_window], may be null                          */
  int32_t* block_len;   /* device [batch], required                                         */
} dc_boundary_out;

typedef struct dc_select_in {
  int32_t batch;
  const float* conf;        /* device [batch][max_window]                                   */
  const int32_t* win_ids;   /* device [batch][max_window]; candidates are == mask_id        */
  const float* xlogp;       /* device [batch][max_window][max_window]                       */
  const int32_t* block_len; /* device [batch]: the current block is window[0, block_len)    */
  const int32_t* win_len;   /* host [batch]                                                 */
  int32_t override_thresholds; /* 1: use the three values below instead of the config's     */
  float tau_low, tau_high, gamma;
} dc_select_in;

typedef struct dc_select_out {
  uint8_t* sel_mask;  /* device [batch][max_window] 1 = commit this position                */
  int32_t* sel_idx;   /* device [batch][max_window] selected positions, ascending           */
  int32_t* sel_count; /* device [batch] |S|                                                 */
} dc_select_out;

typedef struct dc_ctx dc_ctx; /* opaque */

/* Create a context: validates the configuration, records the (borrowed) weight pointers, and
 * allocates the workspace for the given capacities on the current CUDA device.
 * cuda_stream: a cudaStream_t (null = the legacy default stream); all work is ordered on it.
 * Tensor-core kernels need dtype bf16, head_dim 128, d_model and d_ff multiples of 128; any
 * other shape runs on the CUDA-core kernels.  Errors: INVALID_ARG, UNSUPPORTED, NOMEM, CUDA.
 * The backbone is the pre-norm transformer the paper's backbones share (Section 5.1). */
DC_API int dc_create(const dc_config* cfg, const dc_weights* w, void* cuda_stream, dc_ctx** out);

/* One block-step (Section 3, Eq. 1-2: predictions for the masked positions of the active block
 * given the decoded context; Section 4.2, Eq. 3-4: I_k, H_k, S_k and the block boundary).
 * Rows fed to the backbone per sequence: the last decoded block followed by the window, at
 * absolute positions ctx_len[b] + r; with DC_STEP_INFLUENCE a second variant with the last
 * block's ids replaced by mask_id runs in the same pass (p_prev).  Every active row attends all
 * ctx_len[b] cached keys and all active rows of its own variant (no causal mask).
 * Errors: INVALID_ARG, SHAPE, CUDA (host side); status[b] (device side). */
DC_API int dc_step(dc_ctx* ctx, const dc_step_in* in, const dc_step_out* out);

/* The boundary rule alone on caller-supplied signals (Section 4.2; cumulative form Section 4.4):
 * smooth, normalise, S_k = I~_k - lambda*H~_k, first negative, clip to [L_min, L_window].
 * dc_step runs the same kernel when DC_STEP_BOUNDARY is set. */
DC_API int dc_boundary(dc_ctx* ctx, const dc_boundary_in* in, const dc_boundary_out* out);

/* CAP-Decoding (Section 4.3, Eq. 5-6, Algorithm 1): candidate pool, pairwise conflicts,
 * high-confidence phase, greedy completion, single-token fallback.  Reads the buffers a
 * previous dc_step wrote (or any caller-made ones). */
DC_API int dc_select(dc_ctx* ctx, const dc_select_in* in, const dc_select_out* out);

/* The two decision kernels over any number of sequences in one call (a serving layer that batches
 * the decisions of many requests; also what bench.py times for their bandwidth number).  Same
 * kernels, same arithmetic and layouts as dc_boundary / dc_select (row pitch max_window of the
 * context), but the per-sequence lengths are DEVICE arrays [batch] and batch is not limited by
 * max_batch.  have_prev may be null (= all 1).  Section 4.2 / 4.4 and Algorithm 1. */
DC_API int dc_boundary_batched(dc_ctx* ctx, int32_t batch, const float* influence, const float* entropy,
                               const int32_t* win_len, const int32_t* remain_len, const int32_t* have_prev,
                               const dc_boundary_out* out);
DC_API int dc_select_batched(dc_ctx* ctx, int32_t batch, const float* conf, const int32_t* win_ids,
                             const float* xlogp, const int32_t* block_len, const int32_t* win_len,
                             const dc_select_out* out);

/* ---- the decoding loop around the step (Section 3, Eq. 1-2; forward scan of Section 4.2) ----- */

/* Prefill: the K / V of n_ids[b] clean tokens per sequence (a prompt, or any run of decoded
 * tokens whose cache is to be rebuilt), computed by one bidirectional pass over those tokens - they
 * attend one another and the ctx_len[b] keys already in the cache (Section 3: the DLM attends the
 * whole known sequence; block-wise cache reuse, Section 4.1) -
 * and written into the caches at keys ctx_len[b] .. ctx_len[b] + n_ids[b] - 1, every layer.  The
 * same kernels as dc_step without window rows; no LM head.  A prompt goes through in one call
 * (the pass is bidirectional, so chunks would not see each other): n_ids[b] <= max_last and
 * ctx_len[b] + n_ids[b] <= max_ctx, DC_ERR_SHAPE otherwise.  Asynchronous on the handle's stream. */
typedef struct dc_prefill_in {
  int32_t batch;
  void* k_cache;             /* device, layouts as in dc_step, written                        */
  void* v_cache;             /* device, written                                               */
  const int32_t* ctx_len;    /* host [batch], may be null (all 0)                             */
  const int32_t* ids;        /* device [batch][max_last]                                      */
  const int32_t* n_ids;      /* host [batch]                                                  */
  const int32_t* pos0;       /* host [batch] or null: absolute position of ids[b][0]; null means
                                ctx_len[b] (the tokens follow the cached ones).  Other values are
                                for cached rows that do not follow the context in the sequence -
                                the still masked suffix behind the window that a dual cache keeps
                                (Section 5.2, cache compatibility): K is stored rotated, so the
                                position is all a later step needs to know about such a row      */
} dc_prefill_in;
typedef struct dc_prefill_out {
  int32_t* status;           /* device [batch]                                                */
} dc_prefill_out;
DC_API int dc_prefill(dc_ctx* ctx, const dc_prefill_in* in, const dc_prefill_out* out);

/* Eq. (2): y_i <- yhat_i for the selected, still masked positions of the current block
 * window[0, block_len); remaining[b] = masked positions left in that block. */
typedef struct dc_commit_in {
  int32_t batch;
  int32_t* win_ids;          /* device [batch][max_window], updated in place                  */
  const int32_t* pred_id;    /* device [batch][max_window]                                    */
  const uint8_t* sel_mask;   /* device [batch][max_window]                                    */
  const int32_t* block_len;  /* device [batch]                                                */
  const int32_t* win_len;    /* host [batch]                                                  */
} dc_commit_in;
typedef struct dc_commit_out {
  int32_t* remaining;        /* device [batch], may be null                                   */
} dc_commit_out;
DC_API int dc_commit(dc_ctx* ctx, const dc_commit_in* in, const dc_commit_out* out);

/* Block-wise generation of gen_len tokens per sequence after a cached context, with DepCap's two
 * decisions at every stage.  Per sequence, repeated until gen_len tokens are decoded:
 *   boundary step   dc_step over [last decoded block ; L_window masked positions] with the prev
 *                   variant: I_k, H_k -> next block length L (first block: L = L_min); the last
 *                   block's K / V are appended to the cache (DC_STEP_EXPORT_KV); the step's own
 *                   predictions already serve the block: dc_select + dc_commit on [0, L)
 *   denoising steps dc_step over the block's L positions (no prev variant), dc_select,
 *                   dc_commit, until the block holds no [MASK]
 * The host reads block lengths and remaining-mask counts after every step (one small copy and a
 * stream synchronisation per step).  Sequences advance independently; finished ones idle.
 * k_cache / v_cache: as in dc_step, holding ctx_len[b] keys of context on entry, with room for
 * ctx_len[b] + gen_len keys (DC_ERR_SHAPE otherwise); they are extended in place.
 * max_steps bounds the number of dc_step calls (DC_ERR_TIMEOUT when exceeded; <= 0: 4 * gen_len).
 * Prefill of the context is not part of this call. */
typedef struct dc_generate_in {
  int32_t batch;
  void* k_cache;             /* device, written                                               */
  void* v_cache;             /* device, written                                               */
  const int32_t* ctx_len;    /* host [batch]                                                  */
  int32_t gen_len;           /* tokens to decode per sequence, >= 1                           */
  int32_t max_steps;
  int32_t carried_prev;      /* non-zero: boundary steps take p_prev from the rows the boundary
                                step before them left (DC_STEP_CARRIED_PREV) instead of running a
                                second variant                                                */
} dc_generate_in;
typedef struct dc_generate_out {
  int32_t* tokens;           /* HOST [batch][gen_len]                                         */
  int32_t* block_lens;       /* HOST [batch][gen_len]: lengths of the blocks in order, then 0 */
  int32_t* nfe;              /* HOST [1]: dc_step calls made (model forward evaluations)      */
  float* device_ms;          /* HOST [1] or null: summed device time of all forwards (CUDA events
                                around each forward's launches); wall clock minus this is what the
                                host loop and its read-backs cost                              */
} dc_generate_out;
DC_API int dc_generate(dc_ctx* ctx, const dc_generate_in* in, const dc_generate_out* out);

/* Options of a context.  No paper counterpart.
 *   DC_OPT_COOPERATIVE (default 1): the fused dense-layer kernel synchronises its CTAs through a
 *     counter in global memory, which needs all of them resident at once; a cooperative launch
 *     guarantees that (or fails).  0 launches the same grid without the attribute - for profilers
 *     that cannot replay cooperative cluster launches.  All CTAs are still resident when the GPU
 *     runs nothing else, and every wait in the kernel is bounded (DC_ERR_TIMEOUT in status[b]
 *     otherwise), but the guarantee is gone: not for production use.
 *   DC_OPT_WAIT_LIMIT_US (default 2 000 000): how long a device-side wait (on a TMA / MMA
 *     barrier, the grid barrier, a hand-over flag) polls before the kernel gives up, frees what it
 *     holds, returns and reports DC_ERR_TIMEOUT in status[b]; 1000 .. 60 000 000.  The value is
 *     kept on the device and is shared by every context of the process on that device.
 *   DC_OPT_TEST_STALL_LMHEAD (default 0): test hook for the path above.  1 makes the LM-head
 *     kernel skip all of its loads, so that nothing is in flight and every one of its waits runs
 *     out: the step then ends with DC_ERR_TIMEOUT in every status[b] and the context stays usable.
 * Returns DC_ERR_INVALID_ARG for an unknown option or a value out of range. */
enum { DC_OPT_COOPERATIVE = 1, DC_OPT_WAIT_LIMIT_US = 2, DC_OPT_TEST_STALL_LMHEAD = 3 };
DC_API int dc_set_option(dc_ctx* ctx, int32_t option, int32_t value);

/* Frees the workspace.  The caller must have synchronised the stream.  Null is a no-op. */
DC_API int dc_destroy(dc_ctx* ctx);

/* Human-readable reason for the last non-OK return on this context (never null).  With a null
 * context: the reason for the last failed dc_create on this thread. */
DC_API const char* dc_last_error(const dc_ctx* ctx);

/* Debug: copies the curr-variant (variant 0) or prev-variant (1) logits of the last dc_step into
 * out [batch][max_window][vocab] fp32 (device).  Only available when the CUDA-core LM head ran
 * (DC_IMPL_SIMT or an fp32 model); otherwise DC_ERR_UNSUPPORTED.  No paper counterpart. */
DC_API int dc_debug_logits(dc_ctx* ctx, int32_t variant, float* out);

/* Per-stage device time of the last dc_step_profiled call, in milliseconds. */
enum { DC_STAGE_EMBED = 0, DC_STAGE_NORM, DC_STAGE_QKV, DC_STAGE_ATTN, DC_STAGE_OPROJ,
       DC_STAGE_GATEUP, DC_STAGE_DOWN, DC_STAGE_LMHEAD, DC_STAGE_XLOGP, DC_STAGE_BOUNDARY,
       DC_STAGE_DENSE, /* fused launch: O projection, norms, gate/up, down, QKV of the next layer */
       DC_STAGE_COUNT };

/* dc_step with CUDA events around every stage; synchronises the stream before returning and
 * fills stage_ms[DC_STAGE_COUNT] (host) with the summed device time per stage and
 * stage_launches[DC_STAGE_COUNT] (host) with the kernel launches per stage.  For measurement;
 * same results as dc_step.  No paper counterpart. */
DC_API int dc_step_profiled(dc_ctx* ctx, const dc_step_in* in, const dc_step_out* out, float* stage_ms,
                     int32_t* stage_launches);

/* ---- LM-head signals without any allocation -------------------------------------------------
 * The paper has no counterpart of this call; it exists for hosts that must not allocate.
 *
 * Some callers cannot reach cudaMalloc at the moment they need the per-position signals: code
 * that runs inside another framework's memory pool and is forbidden to go around it, code on a
 * latency path where an allocation (an implicit device synchronisation) is not acceptable, or a
 * process whose memory budget was handed out in full at start-up.  dc_create allocates a
 * workspace, so it is closed to them.  dc_signals_static computes what the LM-head stage of
 * dc_step computes - yhat_k, c_k, H_k, I_k and the log-sum-exp for every window position, from
 * LM-head inputs the caller already holds - and keeps its scratch data (the LM-head inputs in
 * the kernel's row order, the per-CTA partial softmax records, a status word) in a fixed array
 * that is part of the library image: DC_STATIC_SCRATCH_BYTES of device memory on every GPU that
 * loads the library, held until the process exits.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine.
 *
 * Limits (DC_ERR_SHAPE / DC_ERR_UNSUPPORTED beyond them, nothing is launched, and
 * dc_last_error(NULL) gives the reason): bf16 only,
 * d_model a multiple of 128 and <= DC_STATIC_MAX_D, batch * round16(longest window) <=
 * DC_STATIC_MAX_POS positions, vocab >= 2.
 *
 * The first call on a device looks up the device address of the array and opts the kernel in to
 * its shared memory; make that first call before any stream capture, and from one host thread
 * (the per-device address table is filled without a lock; later calls only read it).  All calls on a device
 * share the one array, which keeps the previous call's contents: the call itself clears what
 * must start at zero, but two calls whose kernels overlap on the GPU (different streams, no
 * dependency) race on it - order them.  The caller passes inputs and outputs as usual; outputs
 * are valid after the stream is synchronised.  With the same inputs the results are those of
 * dc_step (same kernels, same tiling). */
enum { DC_STATIC_MAX_D = 8192, DC_STATIC_MAX_POS = 128,
       DC_STATIC_SCRATCH_BYTES = 2 * DC_STATIC_MAX_POS * DC_STATIC_MAX_D * 2 /* inputs, bf16 */
                                 + 2 * 160 * 128 * 8 * 4                      /* partial records */
                                 + 4096 /* per-position results, status */ };

typedef struct dc_signals_in {
  int32_t d_model, vocab, mask_id;
  int32_t forbid_mask_pred;  /* 1: [MASK] is removed from both softmaxes                     */
  int32_t batch;             /* sequences, >= 1                                              */
  int32_t max_window;        /* row pitch of h and of the outputs, multiple of 16            */
  const void* lm_head;       /* device bf16 [vocab, d_model], 16-byte aligned                */
  const void* h;             /* device bf16 [batch][2][max_window][d_model]: LM-head input   */
                             /* rows of the curr (0) and prev (1) variant                    */
  const int32_t* win_len;    /* host [batch], 1..max_window                                  */
  const int32_t* have_prev;  /* host [batch] or null (= all 1); 0: I_k is reported as 0      */
} dc_signals_in;

typedef struct dc_signals_out {   /* device, [batch][max_window]; any but status may be null */
  int32_t* pred_id;
  float *conf, *entropy, *influence, *lse;
  int32_t* status;                /* [batch], required: DC_OK, DC_ERR_TIMEOUT or DC_ERR_NUMERIC */
} dc_signals_out;

DC_API int dc_signals_static(const dc_signals_in* in, const dc_signals_out* out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DEPCAP_H_ */
