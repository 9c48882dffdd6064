/* ada.h -- C ABI of the adaptive speculative-decoding iteration (AdaEAGLE) for one B200.
 *
 * One iteration = predict a draft length n with the Lightweight Draft Length
 * Predictor (Eq. 3), draft n tokens with the EAGLE head as a chain (Eq. 2),
 * verify the n+1 candidate positions with the target in one pass over its KV
 * cache (Eq. 1), accept the longest correct prefix plus one bonus token, and
 * roll the caches back to the accepted length (Algorithm 1).
 *
 * Conventions
 *  - Every pointer named d_* is DEVICE memory, everything else is host memory.
 *  - The caller owns weights, workspace and all I/O buffers; they are borrowed
 *    for the lifetime of the context.  The library allocates no device memory.
 *  - Weights are bf16, row-major [out][in].  Token ids and lengths are int32.
 *  - All calls enqueue on the stream given to ada_init and return without
 *    synchronising, except ada_get_counters and ada_destroy.
 *  - Return value: 0 or a negative ADA_ERR_* code.  Argument errors are found on
 *    the host before anything is launched.  Device-side range errors (cache full)
 *    set a status word that ada_get_counters reports; the offending rows are skipped.
 *  - Sequences of a batch are independent; per-sequence arrays are indexed [seq].
 *  - Calling ada_ldlp_predict, ada_draft, ada_verify, ada_accept in that order
 *    gives exactly what one ada_step gives.
 */
#ifndef ADA_H
#define ADA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ADA_OK 0
#define ADA_ERR_BAD_CONFIG (-1)
#define ADA_ERR_NULL (-2)
#define ADA_ERR_RANGE (-3)
#define ADA_ERR_KV_FULL (-4)
#define ADA_ERR_CUDA (-5)
#define ADA_ERR_WORKSPACE (-6)
#define ADA_ERR_STATE (-7)     /* the call cannot run in the context's present state (ada_last_error says why) */
#define ADA_ERR_TOO_LARGE (-8) /* a size exceeds a fixed maximum of the library (see ada_ldlp_eval_static) */

#define ADA_MAX_LAYERS 128
#define ADA_MAX_BATCH 8
#define ADA_MAX_NMAX 15

typedef struct ada_ctx ada_ctx; /* opaque, host memory, owned by the library */

typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  float rope_theta, rms_eps;
  int32_t ldlp_hidden;  /* hidden width of the predictor MLP */
  int32_t n_max;        /* largest draft length (k_max of Eq. 3), 1..15 */
  int32_t ldlp_mode;    /* 0: class logits, n = argmax + 1 (the classification variant of Section 4.3.2);
                         * 1: one scalar, n = clip(round(z), k_min, n_max) (Eq. 3; ties round to even)      */
  int32_t max_batch;    /* sequences decoded together, 1..8 */
  int32_t kv_capacity;  /* positions per sequence, multiple of page_size */
  int32_t page_size;    /* KV page length in positions: 64 */
  int32_t ldlp_blocks;  /* ldlp_mode 1: residual blocks h += ReLU(W_r h + b_r) between the two linear maps, 0..8 */
  int32_t k_min;        /* ldlp_mode 1: smallest draft length (k_min of Eq. 3), 1..n_max                         */
  float ddd_threshold;  /* < 0: the combined stopping rule of Section 4 (AdaEAGLE-DDD): the head keeps drafting past
                         * the predicted length while the log-probability of the draft sequence (sum of the log
                         * softmax probabilities of its tokens) is at or above this value, up to n_max; it stops as
                         * soon as step >= n and log-probability < threshold.  >= 0: off.  Needs max_batch = 1.   */
} ada_config;

/* Device pointers to bf16 tensors.  Per-layer members are HOST arrays of n_layers device pointers. */
typedef struct {
  const void *embed;      /* [vocab][d]  shared by target, draft head and predictor        */
  const void *lm_head;    /* [vocab][d]  shared by target and draft head (Section 2.2)     */
  const void *final_norm; /* [d]                                                            */
  const void *const *wq, *const *wk, *const *wv, *const *wo;   /* [d][d]                    */
  const void *const *w_gate, *const *w_up;                     /* [d_ffn][d]                */
  const void *const *w_down;                                   /* [d][d_ffn]                */
  const void *const *norm_attn, *const *norm_mlp;              /* [d]                       */
  const void *eagle_fc;   /* [d][2d], input [embedding ; feature]                           */
  const void *e_wq, *e_wk, *e_wv, *e_wo, *e_gate, *e_up, *e_down, *e_norm_attn, *e_norm_mlp;
  const void *ldlp_w1, *ldlp_b1; /* [hid][2d], [hid]   input [embedding ; feature] (Section 3.3) */
  const void *ldlp_w2, *ldlp_b2; /* [n_max][hid], [n_max]   (ldlp_mode 1 reads row 0 and entry 0 only) */
  const void *ldlp_wr, *ldlp_br; /* ldlp_mode 1: [ldlp_blocks][hid][hid], [ldlp_blocks][hid]; else unused (may be NULL) */
} ada_weights;

/* Bytes of device workspace (KV pools, feature rows, scratch) ada_init needs for this config;
 * 0 if the config is invalid. */
size_t ada_workspace_bytes(const ada_config *cfg);

/* Validates cfg, carves d_workspace (256-byte aligned, >= ada_workspace_bytes) and builds the
 * rotary table.  cuda_stream is a cudaStream_t (NULL = default stream).
 * With max_batch = 1 every decode pass (draft step, verify) is one persistent kernel launched
 * cooperatively in thread-block clusters of two, one CTA per SM; ada_init checks that the whole grid
 * can be resident and uses the multi-kernel path otherwise.  Batches (max_batch > 1: that kernel's
 * attention reads one sequence's cache) and the prompt of every engine, 128 rows at a time, run the
 * multi-kernel path with its tensor-core GEMM, whose weight boxes are 128 rows high: d_model, d_ffn and
 * vocab must be at least 128 (ADA_ERR_BAD_CONFIG otherwise).  The environment variable ADA_PASS_NONCOOP
 * (any value) drops the cooperative launch attribute, for profilers that refuse it together with
 * clusters. */
int ada_init(ada_ctx **out, const ada_config *cfg, const ada_weights *w, void *d_workspace,
             size_t workspace_bytes, void *cuda_stream);

/* Algorithm 1, first pass (draft length 0): the target reads the m prompt tokens of sequence
 * `seq` (in chunks of up to 128 positions), fills its cache and emits the first new token, which
 * becomes the pending token; the draft head is brought up to date on prompt positions 0..m-2.  d_first_token (optional)
 * receives that token.  1 <= m, m + n_max + 2 <= kv_capacity. */
int ada_prefill(ada_ctx *ctx, int seq, const int32_t *d_prompt, int32_t m, int32_t *d_first_token);

/* Eq. 3: n[seq] = predictor([e ; f]) of the last token of the validated prefix (the token before
 * the pending one) for every sequence; n in [1, n_max], clipped so that n+1 rows fit the cache.
 * An override installed by ada_force_n replaces the prediction.  d_n: [max_batch]. */
int ada_ldlp_predict(ada_ctx *ctx, int32_t *d_n);

/* Eq. 2: the draft head emits d_n[seq] tokens per sequence as a chain (first bringing its cache
 * up to date with the target features of the positions accepted last time).
 * d_draft: [max_batch][n_max], entries beyond n are left untouched. */
int ada_draft(ada_ctx *ctx, const int32_t *d_n, int32_t *d_draft);

/* Label of Section 3.3 (the optimal draft length that the predictor is trained on; the draft-length oracle of
 * Section 2.3 is a decoder that is told it): for every sequence drafts as many tokens as allowed (n_max, or what
 * the cache still holds), verifies them and writes to d_k[seq] the length of the longest prefix of the draft that
 * the target confirms.  Nothing is committed: a following ada_step or ada_draft starts from the same state (the
 * draft head recomputes the row of the last verified position).  d_k: [max_batch]. */
int ada_label(ada_ctx *ctx, int32_t *d_k);

/* Labels for a range of start positions of an already decoded sequence (Section 3.3, data collection: for every
 * position j of a target output, k^j = the length of the longest common prefix of a k_max-token draft started at j and
 * the target's own continuation).  For j = j0 .. j0 + count - 1, with token j of sequence `seq` taken as the pending
 * token and tokens 0..j as the committed prefix, the draft head drafts n_max tokens (fewer at the end of the cache), the
 * target verifies them, and d_k[j - j0] receives the accepted length; d_drafts [count][n_max] and d_targets
 * [count][n_max+1] (optional) receive the drafts and the target's choices, -1 past the draft length.  The positions
 * run one after another, last first, each through the draft and verify kernels of the decode iteration; afterwards
 * the cache rows and features from j0 on are recomputed from the committed tokens (multi-row chunks), so the sequence
 * continues exactly as if the call had not been made.  1 <= j0, j0 + count - 1 <= index of the pending token; the
 * draft head must be up to date (the sequence was decoded with drafts): ADA_ERR_STATE otherwise.  Teacher forcing
 * (ada_force_draft) applies as in ada_label.  This call reads the sequence's length from the device: it synchronises
 * the stream once before it enqueues. */
int ada_label_positions(ada_ctx *ctx, int seq, int32_t j0, int32_t count, int32_t *d_k, int32_t *d_drafts,
                        int32_t *d_targets);

/* The draft lengths in force after ada_draft: d_n itself, or, with ddd_threshold < 0 (Section 4), the lengths
 * the stopping rule settled on; these are the lengths to hand to ada_verify.  d_n: [max_batch]. */
int ada_draft_lengths(ada_ctx *ctx, int32_t *d_n);

/* Eq. 1, forward part: the target runs over the pending token and the n draft tokens of every
 * sequence (n may be 0: plain autoregressive step) and returns its greedy choice after each row.
 * d_target_tok: [max_batch][n_max+1].  d_logits (optional): [max_batch][n_max+1][vocab] fp32. */
int ada_verify(ada_ctx *ctx, const int32_t *d_draft, const int32_t *d_n, int32_t *d_target_tok,
               float *d_logits);

/* Eq. 1, decision part (footnote of Section 3.1) and the roll-back: accept_len = longest draft
 * prefix matching the target's choices; emitted = accepted drafts + bonus token; target cache
 * length and pending token advance; draft cache keeps only rows made from target features.
 * Uses the drafts and target tokens of the last ada_verify.  All outputs optional:
 * d_accept_len [max_batch], d_emitted [max_batch][n_max+1], d_n_emitted [max_batch]. */
int ada_accept(ada_ctx *ctx, int32_t *d_accept_len, int32_t *d_emitted, int32_t *d_n_emitted);

/* One whole iteration of Algorithm 1 (predict -> draft -> verify -> accept) replayed as a
 * captured CUDA graph; draft lengths never visit the host.  Outputs as in ada_accept plus
 * d_n_used [max_batch] (the draft lengths used); all optional. */
int ada_step(ada_ctx *ctx, int32_t *d_emitted, int32_t *d_n_emitted, int32_t *d_n_used,
             int32_t *d_accept_len);

/* Test and measurement hooks ------------------------------------------------------------- */

/* Fixed draft lengths instead of the predictor: n[seq] (host array of max_batch entries, each
 * 0..n_max; 0 = plain autoregressive decoding: the draft head is then not kept up to date, and
 * while every length is forced to 0 ada_draft returns ADA_ERR_STATE; a sequence whose head fell behind by
 * more rows than one pass holds drafts nothing from then on and the status word gets its "stale" bit).
 * NULL restores the predictor. */
int ada_force_n(ada_ctx *ctx, const int32_t *n);

/* Teacher forcing: after every draft step the drafted token of sequence seq is replaced by
 * d_tokens[seq][step] (device, [max_batch][n_max]).  The array is copied (stream-ordered) when the call is
 * made; call again to change the tokens.  NULL switches it off. */
int ada_force_draft(ada_ctx *ctx, const int32_t *d_tokens);

/* Replace the outcome of the iteration that just ran for sequence `seq`: rewind to its start and
 * commit the `count` given tokens instead (count-1 accepted drafts and a bonus token, 1 <= count
 * <= n_max+1), recomputing cache rows and features from them.  Used to keep a run on a reference
 * trajectory. */
int ada_force_commit(ada_ctx *ctx, int seq, const int32_t *d_tokens, int32_t count);

/* Synchronises the stream and returns, summed over sequences:
 * out[0] N_target (verify passes), out[1] N_draft, out[2] N_waste, out[3] tokens emitted
 * (Table 2's counters), out[4] device status word (0 = no device-side error),
 * out[5] kernels launched by this context so far, out[6..7] 0. */
int ada_get_counters(ada_ctx *ctx, int64_t out[8]);

/* Clears the device status word (stream-ordered).  After a device-side error (out[4] of ada_get_counters non-zero)
 * the results of the calls since the last clear are not to be trusted; bit 4 (a bounded wait inside a kernel gave
 * up) also makes every later pass give up its waits at once, so clear it before going on. */
int ada_reset_status(ada_ctx *ctx);

/* Failure detection (no passage of the paper: every wait inside the kernels -- on an mbarrier, on the grid barrier,
 * on the K-split pair's barrier -- is bounded, and gives up by setting bit 4 of the status word and carrying on).
 * This call runs the kernels' own wait routines on a barrier that nothing ever completes, with a limit of
 * spin_limit polls (1 .. 2^22), so that the give-up path can be seen to run: mode 0 waits on an mbarrier phase
 * nobody arrives at, mode 1 on a grid-barrier count that is never reached.  d_result[mode] (device, 2 x int32) is
 * set to 1 when the wait has returned; ada_get_counters then reports status bit 4.  The context stays usable:
 * clear the word with ada_reset_status. */
int ada_selftest_bounded_wait(ada_ctx *ctx, int32_t mode, uint32_t spin_limit, int32_t *d_result);

/* Device pointer and byte size of an internal buffer, for inspection by tests:
 * which = 0 features f [max_batch][kv_capacity][d] fp32 (row = position),
 *         1 predictor outputs z [max_batch][16] fp32, 2 committed tokens [max_batch][kv_capacity] int32,
 *         3 lengths [max_batch][8] int32 (len, draft-cache len, n, accept_len, ...),
 *         4 draft-head features of the last draft call [max_batch][n_max][d] fp32,
 *         5 top-2 logits of every verify row [max_batch][n_max+1][2] fp32,
 *         6 top-2 logits of every draft step [max_batch][n_max][2] fp32,
 *         7 draft tokens of the last draft [max_batch][n_max] int32,
 *         8 target choices of the last verify [max_batch][n_max+1] int32,
 *         9 phase clock of the last profiled target pass (batch 1, ada_profile on): 512 uint64
 *           nanosecond stamps, [0] = start, [i+1] = end of phase i (embedding, then per layer
 *           QKV, attention, O, gate/up, down, then the LM head). */
int ada_debug_buffer(ada_ctx *ctx, int which, void **d_ptr, size_t *bytes);

/* Measurement hook for roofline reports.  ada_profile(ctx, 1) clears the records and from then on
 * brackets every GEMM launch and every attention launch pair of the separately called steps
 * (not of the ada_step graph) with CUDA events on the context's stream; ada_profile(ctx, 0) stops.
 * ada_get_profile synchronises and returns out[0] GEMM launches, out[1] their summed duration (ms),
 * out[2] the weight bytes they streamed (each weight once per launch), out[3] attention launch
 * pairs, out[4] their summed duration (ms), out[5..7] 0.  At most 4096 launches are recorded. */
int ada_profile(ada_ctx *ctx, int enable);
int ada_get_profile(ada_ctx *ctx, double out[8]);

/* Length predictor for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a packaging variant of ada_ldlp_predict, not a step of the method).
 * Every other call runs inside a workspace that the caller allocated; this one needs none.  It is
 * meant for code that cannot call cudaMalloc at all: a plugin inside a host application that owns
 * all device memory, code running while another allocator holds the whole GPU, or a latency-bound
 * path where an allocation would stall the device.  Its only scratch, the predictor's hidden
 * activations, lives in a fixed array inside the library image: ADA_STATIC_MAX_HIDDEN floats
 * (16 KiB) on every GPU that loads the library, until the process exits.
 *   z = W2 ReLU(W1 [e ; f] + b1) + b2,  n = argmax(z) + 1 (lowest index among equals)
 * d_w1 [hidden][2*d_model], d_b1 [hidden], d_w2 [n_max][hidden], d_b2 [n_max], d_embed_row [d_model]
 * are bf16; d_feature [d_model] fp32; outputs d_n (one int32) and d_z ([n_max] fp32, optional).
 * All pointers are device memory owned by the caller; the call enqueues on cuda_stream and returns.
 * No override and no cache-capacity clip are applied (there is no context).
 * Errors: ADA_ERR_TOO_LARGE if hidden > ADA_STATIC_MAX_HIDDEN (nothing is launched),
 * ADA_ERR_RANGE for other bad sizes, ADA_ERR_NULL, ADA_ERR_CUDA.
 * The first call on each device looks up the array's device address (that device must be current);
 * make that first call before any stream capture begins.  All calls on a device share the array,
 * which keeps the previous call's contents (nothing in it needs clearing: each call overwrites
 * what it reads); calls that overlap on the GPU race on it, so order them on one stream. */
#define ADA_STATIC_MAX_HIDDEN 4096
int ada_ldlp_eval_static(const void *d_w1, const void *d_b1, const void *d_w2, const void *d_b2,
                         const void *d_embed_row, const float *d_feature, int32_t d_model, int32_t hidden,
                         int32_t n_max, int32_t *d_n, float *d_z, void *cuda_stream);

/* Text of the last host-side error of this context ("" if none). */
const char *ada_last_error(const ada_ctx *ctx);

int ada_destroy(ada_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* ADA_H */
