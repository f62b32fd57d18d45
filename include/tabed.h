/*
 * tabed.h - C boundary of the B200 TABED speculative-decoding library.
 *
 * One speculative-decoding round of Test-time Adaptive Batched Ensemble Drafting:
 *   Algorithm 1 (batched shared-weight drafting of m inputs for gamma steps, weighted-average
 *   ensemble and Sample at every step), the verification of Sec. 3 item 3 (accept with
 *   probability min(1, p/q), resample the first rejected token from norm(max(0, p - q))), and
 *   the test-time weight adaptation of Sec. 4.1 / App. B (deviation of each drafter from the
 *   target over a window of h verified positions -> next block's ensemble weights).
 *
 * Conventions
 *   - Every function returns TABED_OK (0) or a negative TABED_ERR_* code; nothing throws, aborts
 *     or prints.  tabed_strerror() names a code.
 *   - Unless a parameter says "host", array arguments are DEVICE pointers on config.device.
 *     Work is enqueued on config.stream and the call returns without synchronising the host;
 *     results are valid once the caller has synchronised that stream.  The *_host entry points
 *     take HOST pointers, copy in, run, copy out and synchronise.
 *   - The caller owns weights, inputs and outputs (weights must outlive the handle).  The library
 *     owns KV caches, the window ring, the per-round q / q^(k) / p buffers and all scratch, all
 *     allocated in tabed_init and released in tabed_destroy; no call in between allocates.
 *   - Alignment: every drafter weight pointer (tabed_weights) must be 16-byte aligned (the projection
 *     kernels read them with 128-bit loads; tabed_init rejects others with TABED_ERR_INVALID_ARG).
 *     Other array arguments need only their element's natural alignment: 16-byte aligned pointers
 *     take the 128-bit paths, others (e.g. offset views) the element-wise ones, with identical results.
 *   - Device-side failures (a bounded wait that ran out, a cache position beyond kv_capacity, a
 *     distribution without mass) set bits in an error word on the device.  tabed_round_host, which
 *     synchronises anyway, returns the matching code (TABED_ERR_TIMEOUT / _KV_OVERFLOW / _NUMERIC) and
 *     clears the word; after the asynchronous calls use tabed_last_device_error.
 *   - Layouts are row-major with the last index fastest.  B = n_requests, m = n_inputs,
 *     R = B*m rows (row = request*m + input), V = vocab, G = gamma.
 *   - Uniforms are caller-supplied floats on the lattice u = (k + 1/2) * 2^-23, 0 <= k < 2^23.
 *   - Per round the order is fixed: draft (tabed_draft_round or tabed_draft_round_logits) ->
 *     tabed_verify -> tabed_update_weights; anything else returns TABED_ERR_BAD_STATE.
 *   - Integer outputs (tokens, accept counts, weight argmax) are functions of the fp32 logits
 *     evaluated with order-independent arithmetic: every floating-point step is one correctly
 *     rounded binary32 operation and every vocabulary-wide sum is a sum of integers
 *     (masses trunc(q_v * 2^40)), so they do not depend on grid shape or scheduling.
 */
#ifndef TABED_H
#define TABED_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TABED_OK                0
#define TABED_ERR_INVALID_ARG  -1
#define TABED_ERR_NULL_PTR     -2
#define TABED_ERR_BAD_STATE    -3
#define TABED_ERR_KV_OVERFLOW  -4
#define TABED_ERR_CUDA         -5
#define TABED_ERR_TIMEOUT      -6
#define TABED_ERR_UNSUPPORTED  -7
#define TABED_ERR_NUMERIC      -8   /* a distribution had no mass to draw from (non-finite logits) */

#define TABED_DTYPE_FP32 0      /* fp32 weights and KV cache, no intermediate rounding          */
#define TABED_DTYPE_BF16 1      /* bf16 weights and KV cache, fp32 accumulation, matmul inputs
                                   rounded to bf16 (nearest even)                               */

#define TABED_POLICY_STATIC          0   /* w_k = 1/m (the paper's Static baseline)              */
#define TABED_POLICY_GRID_MT         1   /* m = 2: w^j = [1-j/10, j/10], j = 0..10, argmin error  */
#define TABED_POLICY_SOFTMAX_INV_ERR 2   /* w = softmax(1/e^(1..m); tau)                          */
#define TABED_POLICY_RANDOM          3   /* ablation of Sec. 5 ("Effectiveness of Dynamic Weights"): non-negative
                                            sum-to-one random weights, a uniform point of the simplex drawn from
                                            caller-supplied uniforms (tabed_set_policy_uniforms)     */
#define TABED_POLICY_GRID_HARD       4   /* m = 2, hard labels (Sec. 4.1): the grid candidate whose most likely
                                            token matched the verified token most often in the window  */
#define TABED_POLICY_ADABOOST        5   /* appendix "TABED-AdaBoost": w_k = ln(1/eps_k - 1) + C ln(V - 1),
                                            eps_k = (errors_k + 1) / (n + 2) over the n window positions (an error:
                                            the drafter's most likely token is not the verified token), negative
                                            values cut at 0, normalised; C = config.tau                */

#define TABED_DIST_KL   0       /* D = KL(p || q)        */
#define TABED_DIST_TVD  1       /* D = 1/2 sum |p - q|   */

#define TABED_MODE_SAMPLE 0     /* tokens drawn from q with the supplied uniforms */
#define TABED_MODE_GREEDY 1     /* argmax decoding, lowest id on ties             */

#define TABED_MAX_INPUTS 8
#define TABED_MAX_TREE_WIDTH 4

/* Token tree of width d (Sec. 5, "Verification: Integrating Token Tree"; config.tree_width = d > 1).  The paper names the
 * method and the widths 2 and 3; the construction taken here: at every depth of the block the drafter proposes d
 * distinct candidates, drawn from the ensembled q WITHOUT replacement (greedy mode: its d most likely tokens); the
 * first one (the primary) is the token the chain continues with, the others are leaves.  The target scores the chain
 * and every leaf in one pass (G + 1 + G (d - 1) rows).  At the first depth whose primary is rejected the siblings are
 * tried in order by recursive rejection: after a rejection p' = norm(max(0, p' - q')), q' = q' restricted to the
 * untried tokens, renormalised; candidate x is accepted iff p'(x) >= q'(x) or u q'(x) < p'(x); if all are rejected the
 * replacement is drawn from the last residual.  An accepted sibling ends the block; the next token then comes from the
 * target's distribution at its leaf.  The emitted tokens follow the target's law as in Sec. 3.  Shapes with d > 1:
 * u_draft, out_tokens, u_accept are [B][G][d] (candidate-minor; column 0 = the primary chain); target_logits is
 * [B][G + 1 + G (d - 1)][V]: rows 0..G the chain's positions, row G + 1 + i (d - 1) + (c - 1) the leaf after sibling c of
 * depth i.  n_accept counts an accepted sibling too.  d = 1 is exactly the plain round.  With d > 1 drafting runs on
 * the tensor-core or per-operation path. */

/* tabed_debug_view selectors (device buffers owned by the handle) */
#define TABED_VIEW_QK          0   /* float  [B][G][m][V]  per-drafter distributions of the round     */
#define TABED_VIEW_Q           1   /* float  [B][G][V]     ensembled distributions of the round        */
#define TABED_VIEW_P           2   /* float  [B][G+1][V]   target distributions (after tabed_verify); with a token tree
                                                           [B][G+1+G(d-1)][V], of the leaves only the one that was used */
#define TABED_VIEW_LOGITS      3   /* float  [G][B][m][V]  drafter logits of the round's own forward   */
#define TABED_VIEW_KV_LEN      4   /* int32  [R]           committed cache length of every row         */
#define TABED_VIEW_WEIGHTS     5   /* float  [B][m]        current ensemble weights w*                 */
#define TABED_VIEW_WINDOW_SUM  6   /* int64  [B][n_dev]    windowed deviation, fixed point 2^-40 (KL)
                                                           or 2^-41 (TVD); n_dev = 11 (grid) or m     */
#define TABED_VIEW_PENDING     7   /* int32  [B][3]        {count, token0, token1}                     */
#define TABED_VIEW_GRID_J      8   /* int32  [B]           j* of the grid policy (-1 before any update)*/
#define TABED_VIEW_ERROR_FLAG  9   /* int32  [1]           non-zero if a device-side check failed      */
#define TABED_VIEW_ACC_PRIMARY 11  /* int32  [B]           accepted tokens of the primary chain (after tabed_verify)   */
#define TABED_VIEW_SIBLING     12  /* int32  [B]           token of the accepted sibling of a token tree, or -1        */
#define TABED_VIEW_TRACE      10   /* uint64 [G][5L+8][8]  phase timeline of the persistent drafting kernel
                                                           (tabed_debug_trace): one record per phase */

/* How tabed_draft_round runs Algorithm 1 (tabed_select_path).  Results obey the same contract on
 * every path: identical integer decisions for identical logits; logits agree within the forward
 * pass's floating-point tolerance (summation order differs).  The selection also governs how
 * tabed_prefill_* feed a prompt: with TABED_PATH_PER_OP one position at a time, otherwise (bf16
 * drafter) in chunks of 256 positions through the tensor-core kernels. */
#define TABED_PATH_AUTO        0   /* persistent kernel if the drafter qualifies, else tensor-core
                                      projections if it qualifies, else per-operation                    */
#define TABED_PATH_PER_OP      1   /* one kernel per operation (any drafter, any number of rows)        */
#define TABED_PATH_PERSISTENT  2   /* the whole round in one cooperative kernel: bf16 drafter, tree_width 1,
                                      B*m <= 8 rows (with more than 4 rows at least two layers: the first of
                                      two pending tokens then gets a weight pass of its own), d_model <= 2048
                                      (<= 1024 with more than 4 slots: 3 - 4 or 5 - 8 rows) and
                                      a multiple of 16, d_ffn a multiple of 16, H <= 64, (H/Hkv)*head_dim <= 512, <= 64 layers,
                                      kv_capacity <= 32768                                                */
#define TABED_PATH_TENSOR_CORE 3   /* one kernel per operation with the projections as tcgen05 contractions
                                      over all rows: any bf16 drafter with d_model, d_ffn, H*head_dim
                                      multiples of 8 (the automatic choice when the persistent kernel
                                      does not take the shape, i.e. more than 8 rows)                     */

typedef struct tabed_handle tabed_handle;   /* opaque, library-owned */

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, d_ffn, vocab;
  int32_t dtype;              /* TABED_DTYPE_* */
  float   rms_eps;            /* e.g. 1e-5 */
  float   rope_theta;         /* e.g. 10000 */
  int32_t n_inputs;           /* m: drafting inputs per request, 1..TABED_MAX_INPUTS */
  int32_t n_requests;         /* B >= 1 */
  int32_t gamma;              /* block length, 1..16 */
  int32_t window_h;           /* h; 0 = ALL (unbounded running sum) ; <= 64 */
  int32_t policy;             /* TABED_POLICY_* */
  int32_t distance;           /* TABED_DIST_* */
  int32_t sample_mode;        /* TABED_MODE_* */
  float   tau;                /* temperature of TABED_POLICY_SOFTMAX_INV_ERR; constant C of TABED_POLICY_ADABOOST; > 0 */
  int32_t kv_capacity;        /* tokens per row */
  int32_t device;             /* CUDA device ordinal */
  void*   stream;             /* cudaStream_t, caller-owned; NULL = legacy default stream */
  int32_t tree_width;         /* d: candidates per depth of the token tree, 1..TABED_MAX_TREE_WIDTH; 0 or 1 = a plain chain */
} tabed_config;

/* Device pointers to the drafter M_q, element type per config.dtype (float or bf16), every matrix
 * [out][in] row-major; per-layer arrays are HOST arrays of n_layers device pointers.
 * wq [d][d], wk/wv [Hkv*hd][d], wo [d][d], w_gate/w_up [F][d], w_down [d][F], norms [d],
 * embed [V][d], lm_head [V][d] (untied), final_norm [d].  A NULL drafter (weights == NULL in
 * tabed_init) gives a handle on which only the logits-driven calls are available. */
typedef struct {
  const void *embed, *lm_head, *final_norm;
  const void *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *w_gate, *const *w_up, *const *w_down;
  const void *const *norm1, *const *norm2;
} tabed_weights;

/* Create a handle: validates the configuration, allocates every library-owned buffer, sets the
 * ensemble weights to 1/m (no history yet) and leaves every row cache empty.
 * Errors: NULL_PTR, INVALID_ARG (sizes out of range, head_dim not in {32,64,128}, d_model or
 * d_ffn not a multiple of 8, a grid policy with m != 2, a weight pointer that is not 16-byte aligned),
 * UNSUPPORTED, CUDA (allocation failed). */
int tabed_init(const tabed_config* cfg, const tabed_weights* weights, tabed_handle** out);

/* Release everything tabed_init allocated.  NULL is accepted. */
void tabed_destroy(tabed_handle* h);

const char* tabed_strerror(int code);

/* Load a synthetic cache into one row: k, v are [L][Hkv][len][hd] in the drafter's dtype;
 * sets the row's committed length to len.  Errors: INVALID_ARG (row / len out of range). */
int tabed_load_prefix_kv(tabed_handle* h, int32_t row, const void* k, const void* v, int32_t len);

/* Consume a prompt prefix into one row's cache by running the drafter over it (Algorithm 1's
 * prefix x^(k)): causal attention, position by position or in chunks of positions (see TABED_PATH_*).  tokens: int32 [len]; embeds: float [len][d] (projected
 * image tokens enter as embeddings).  Appends at the row's committed length.
 * Errors: INVALID_ARG, KV_OVERFLOW, BAD_STATE (handle without drafter). */
int tabed_prefill_tokens(tabed_handle* h, int32_t row, const int32_t* tokens, int32_t len);
int tabed_prefill_embeds(tabed_handle* h, int32_t row, const float* embeds, int32_t len);

/* Pooled multimodal drafting input (Sec. 5, "Pooled Multimodal Drafting (P)"): the visual tokens of one image,
 * in: float [grid_h * grid_w][d] on the device (row-major 2-D arrangement, 24 x 24 in the paper's default), are
 * averaged over every 2 x 2 block of tokens, feature by feature: out float [(grid_h/2) * (grid_w/2)][d] on the
 * device (576 -> 144 tokens), the correctly rounded mean of the four values.  The caller owns both buffers (they must
 * not be the same); the result is a prefix for tabed_prefill_embeds once it is in the drafter's embedding space.  Runs on the handle's
 * stream.  Errors: NULL_PTR, INVALID_ARG (a grid side odd or < 2, d < 1, in == out). */
int tabed_pool_embeds(tabed_handle* h, const float* in, int32_t grid_h, int32_t grid_w, int32_t d, float* out);

/* Set the verified-but-not-yet-consumed token(s) of every request: tok int32 [B][2],
 * cnt int32 [B] with values 1 or 2.  Normally only needed once, before the first round. */
int tabed_set_pending(tabed_handle* h, const int32_t* tok, const int32_t* cnt);

/* One batched shared-weight decoder step outside a round (Algorithm 1 step 5 alone): feeds
 * tok[b] to all m rows of request b at each row's own position, appends K,V, advances the
 * committed lengths by one, and writes logits float [B][m][V] unless out_logits is NULL (then
 * the LM head is skipped).  Errors: KV_OVERFLOW, BAD_STATE (mid-round or no drafter). */
int tabed_decode_step(tabed_handle* h, const int32_t* tok, float* out_logits);

/* Algorithm 1 steps 6-7 on caller-supplied logits float [B][m][V]: q^(k) = softmax(logits^(k)),
 * q = sum_k w_k q^(k), y = Sample(q; u) (or argmax in greedy mode).  w float [B][m] may be NULL
 * (use the handle's current w*).  u float [B].  Outputs: y int32 [B]; q float [B][V] and
 * qk float [B][m][V] may each be NULL.  Stateless with respect to the round. */
int tabed_ensemble_step(tabed_handle* h, const float* logits, const float* w, const float* u,
                        int32_t* y, float* q, float* qk);

/* Algorithm 1: gamma batched drafting steps with the handle's w*, feeding the pending token(s)
 * first (two pending tokens are consumed in the same weight pass).  u_draft float [B][G].
 * Outputs: out_tokens int32 [B][G]; out_q float [B][G][V] may be NULL (the library keeps its own
 * copy either way).  The rows' caches receive the pending and the first G-1 drafted tokens; the
 * committed lengths do not move until tabed_update_weights.
 * Errors: BAD_STATE, KV_OVERFLOW (conservative host-side bound), NULL_PTR. */
int tabed_draft_round(tabed_handle* h, const float* u_draft, int32_t* out_tokens, float* out_q);

/* The same round on caller-supplied drafter logits float [G][B][m][V] (for callers that run M_q
 * themselves): no forward pass, caches untouched. */
int tabed_draft_round_logits(tabed_handle* h, const float* drafter_logits, const float* u_draft,
                             int32_t* out_tokens, float* out_q);

/* Sec. 3 item 3 on the round just drafted.  target_logits float [B][G+1][V] (position G is the
 * bonus position), u_accept float [B][G], u_resid float [B].  p_i = softmax(target_logits_i);
 * token i is accepted iff p_i(y_i) >= q_i(y_i) or u_i * q_i(y_i) < p_i(y_i), stopping at the first
 * rejection; n_accept = a.  next_token: a < G -> drawn from norm(max(0, p_a - q_a)) (from p_a if
 * that residual has no mass); a == G -> drawn from p_G.  Greedy mode: accept iff
 * argmax p_i == y_i, next_token = argmax p_a.  Outputs int32 [B] each. */
int tabed_verify(tabed_handle* h, const float* target_logits, const float* u_accept,
                 const float* u_resid, int32_t* out_n_accept, int32_t* out_next_token);

/* Sec. 4.1 / App. B on the round just verified: for every verified position i <= min(a, G-1)
 * computes the deviation D(p_i, q_i^(k)) of each drafter (or of each of the 11 grid candidates),
 * pushes it into the request's window of the last h positions, evaluates the policy on the
 * window sums to get the next block's w* (Algorithm 1 steps 2-3), then commits the caches:
 * length += pending + (a < G ? a : G-1), pending <- {next_token} or {y_{G-1}, next_token}.
 * Outputs: out_w float [B][m], out_w_argmax int32 [B] (lowest index on ties); either may be NULL. */
int tabed_update_weights(tabed_handle* h, float* out_w, int32_t* out_w_argmax);

/* Uniforms of TABED_POLICY_RANDOM for the next tabed_update_weights: u_policy float [B][m] on the device, on
 * the uniform lattice; the buffer must stay valid until that call has run.  w_k = g_k / sum_j g_j with
 * g_k = -ln u_k.  tabed_update_weights returns TABED_ERR_BAD_STATE under that policy if none was ever set. */
int tabed_set_policy_uniforms(tabed_handle* h, const float* u_policy);

/* Host-buffer round: tabed_draft_round -> tabed_verify -> tabed_update_weights with HOST pointers
 * (pageable or pinned) for every argument, same shapes as above.  Copies the inputs to the
 * device, runs the round, copies the results back and synchronises the stream before returning.
 * The target's logits (the bulk of the input) are copied on a stream of the library's own while the
 * drafting runs on config.stream; that copy starts after all earlier work on config.stream and the
 * verification waits for it, so the caller sees the ordering of a single stream.
 * out_w and out_w_argmax may be NULL. */
int tabed_round_host(tabed_handle* h, const float* u_draft, const float* u_accept,
                     const float* u_resid, const float* target_logits, int32_t* out_tokens,
                     int32_t* out_n_accept, int32_t* out_next_token, float* out_w,
                     int32_t* out_w_argmax);

/* Synchronises the stream and returns the code of the device-side failures recorded since the last call
 * (TABED_OK if none; TABED_ERR_TIMEOUT: a bounded wait of a kernel ran out, its results are void;
 * TABED_ERR_KV_OVERFLOW: a row reached kv_capacity; TABED_ERR_NUMERIC: a distribution had no mass), then
 * clears the record.  For use after the asynchronous calls, whose return codes only cover the host side. */
int tabed_last_device_error(tabed_handle* h);

/* Reads the rows' committed cache lengths and the pending-token counts back (synchronises the stream) so that
 * the host-side overflow check of tabed_draft_round, which otherwise assumes that every round kept its
 * maximum of gamma + 1 positions per row, works on exact lengths again.  tabed_round_host keeps them exact
 * by itself.  Errors: BAD_STATE (mid-round), CUDA. */
int tabed_sync_lengths(tabed_handle* h);

/* Test aid for the failure path of the device-side waits: launches ONE CTA that waits, with the persistent
 * kernel's own bounded poll, for a flagged word that nobody writes, so that the wait (about 2^21 polls, a
 * fraction of a second) runs out, records the failure and returns by itself - the GPU keeps
 * answering.  Returns what tabed_last_device_error then reports (TABED_ERR_TIMEOUT).
 * Errors: UNSUPPORTED (handle without the persistent kernel), CUDA. */
int tabed_debug_barrier_timeout(tabed_handle* h);

/* Choose the drafting path (TABED_PATH_*).  Errors: UNSUPPORTED (TABED_PATH_PERSISTENT on a drafter
 * that does not qualify; likewise TABED_PATH_TENSOR_CORE), BAD_STATE (mid-round), INVALID_ARG.
 * tabed_current_path returns the path the next tabed_draft_round will take: TABED_PATH_PER_OP,
 * TABED_PATH_PERSISTENT or TABED_PATH_TENSOR_CORE (positive), or a negative error code. */
int tabed_select_path(tabed_handle* h, int32_t path);
int tabed_current_path(const tabed_handle* h);

/* Switch the phase timeline of the persistent kernel off (on = 0) or on (on = 1 + the index of the CTA
 * that records; CTA 0 if the grid is smaller): when on, that CTA stores one record of
 * 8 words per phase into TABED_VIEW_TRACE (first index = drafting step): [0] the GPU's
 * nanosecond timer at the end of the phase; [1..5] SM clock cycles that that CTA spent in the phase
 * waiting for and staging activations, waiting for weight tiles, in the tensor-core products,
 * issuing weight copies and in epilogues, and in the rest (for the phases without weights: all of the
 * phase); [6..7] unused.  Phase order within a step: per layer QKV, attention, O, gate/up, down; then
 * LM head, [1 more when tabed_debug_override_logits is set], exp-sum, mix.
 * Errors: UNSUPPORTED (no persistent path). */
int tabed_debug_trace(tabed_handle* h, int32_t on);

/* Pointer and size of a library-owned device buffer (TABED_VIEW_*).  Read-only for the caller. */
int tabed_debug_view(tabed_handle* h, int32_t what, void** dev_ptr, size_t* bytes);

/* Allocation-free variant of tabed_ensemble_step (the paper has no counterpart: this is a
 * deployment convenience, not a step of the method).
 *
 * For callers that must not allocate device memory at the point of use: a serving process that has
 * already handed the whole GPU to its own memory pool, a plug-in running under a fixed memory
 * budget, or a latency-critical path where cudaMalloc (which may synchronise the device and may
 * fail late) is not acceptable.  Such callers cannot create a handle, because tabed_init allocates.
 * This entry point needs no handle and calls no cudaMalloc / cudaFree or any allocating routine:
 * its scratch (row maxima and sums, per-chunk masses) is a fixed 144 KB array compiled into the
 * library's device image, held by every GPU that loads the library until the process exits.
 *
 * Computes exactly what tabed_ensemble_step computes: q^(k) = softmax(logits^(k)),
 * q = sum_k w_k q^(k), y = Sample(q; u) (argmax when sample_mode is TABED_MODE_GREEDY).
 * Device pointers on `device`: logits float [B][m][V], w float [B][m] (required), u float [B];
 * outputs y int32 [B], q float [B][V] (required: the draw re-reads it), qk float [B][m][V] or NULL.
 * Work is enqueued on `stream` (cudaStream_t, NULL = legacy default stream); no host synchronisation.
 *
 * Limits: B*m <= TABED_STATIC_MAX_ROWS and B*ceil(V/2048) <= TABED_STATIC_MAX_CHUNKS; larger
 * problems return TABED_ERR_UNSUPPORTED (use a handle).  m <= TABED_MAX_INPUTS.
 * The first call on each device looks up the scratch array's device address (a host-side set-up
 * step); make that first call before any stream capture begins.
 * All calls on one device share the one scratch array, which keeps the last call's contents (the
 * call clears what has to start at zero): two calls whose kernels overlap on the GPU, e.g. on
 * different streams, race.  Serialise them on one stream or with events.
 * A distribution without mass (non-finite logits) gives token 0 and is recorded in the scratch array;
 * tabed_static_last_error(device, stream) synchronises that stream, returns TABED_ERR_NUMERIC if one was
 * recorded since its last call (else TABED_OK) and clears the record; it allocates nothing either. */
#define TABED_STATIC_MAX_ROWS   1024
#define TABED_STATIC_MAX_CHUNKS 8192
int tabed_ensemble_step_static(const float* logits, const float* w, const float* u, int32_t n_requests,
                               int32_t n_inputs, int32_t vocab, int32_t sample_mode, int32_t device,
                               void* stream, int32_t* y, float* q, float* qk);
int tabed_static_last_error(int32_t device, void* stream);

/* Stand-alone run of the tensor-core projection used for many shared-weight rows (Sec. 4.1 "batched
 * inference": all rows share the parameters, so a projection is one weights x rows contraction):
 * out[s][o] = sum_k w[o][k] * bf16(act[s][k]), fp32 accumulation.  w bf16 [rows][K], act float [n][K],
 * out float [n][rows], all device pointers on `device`; K a multiple of 8, n <= 256; ks = number of
 * splits of the input dimension (partial sums are added in split order).  Allocates and frees its
 * own temporaries and synchronises the stream: a test and tuning aid, not part of the round.
 * Errors: INVALID_ARG, CUDA, TIMEOUT (a bounded device-side wait ran out). */
int tabed_debug_gemm_tc(const void* w, const float* act, int32_t rows, int32_t K, int32_t n, int32_t ks,
                        float* out, int32_t device, void* stream);

/* Replay aid: while set (non-NULL), tabed_draft_round still runs its own forward pass (caches and
 * TABED_VIEW_LOGITS are written as usual) but steps 6-7 of Algorithm 1 read these logits
 * float [G][B][m][V] instead, so that a recorded trajectory can be followed exactly while the
 * forward pass is compared against it.  The buffer must stay valid until cleared with NULL. */
int tabed_debug_override_logits(tabed_handle* h, const float* drafter_logits);

/* Small host-side snapshot of the adaptive state (weights, window ring, pending tokens, committed
 * lengths); cache contents stay on the device.  Call with host == NULL to get the size in *bytes.
 * Both calls synchronise the stream. */
int tabed_state_export(tabed_handle* h, void* host, size_t* bytes);
int tabed_state_import(tabed_handle* h, const void* host, size_t bytes);

/* Device timing of one kernel class: between tabed_profile_begin and tabed_profile_end the library
 * records a CUDA event pair on config.stream around every launch (group) of that class;
 * tabed_profile_end synchronises the stream and returns the summed elapsed milliseconds and the
 * number of timed intervals.  TABED_PROF_ATTENTION, _ENSEMBLE, _VERIFY and _UPDATE time their group
 * of kernels as one interval; the others time a single kernel per interval.  Classes 0-6 only occur
 * on the per-operation path, TABED_PROF_DRAFT_ROUND only on the persistent path. */
#define TABED_PROF_QKV        0
#define TABED_PROF_ATTENTION  1
#define TABED_PROF_OPROJ      2
#define TABED_PROF_GATEUP     3
#define TABED_PROF_DOWN       4
#define TABED_PROF_LM_HEAD    5
#define TABED_PROF_ENSEMBLE   6
#define TABED_PROF_VERIFY     7
#define TABED_PROF_UPDATE     8
#define TABED_PROF_DRAFT_ROUND 9  /* the persistent kernel: one interval per tabed_draft_round */
int tabed_profile_begin(tabed_handle* h, int32_t kernel_class);
int tabed_profile_end(tabed_handle* h, double* total_ms, int64_t* n_intervals);

/* Number of kernels the library has launched on this handle since tabed_init (host counter). */
int64_t tabed_launch_count(const tabed_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* TABED_H */
