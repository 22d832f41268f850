/*
 * pvlm.h - C ABI of the per-step verify / prune / accept hot path of a
 * draft-then-verify (speculative decoding) loop for Video-LLMs, for NVIDIA
 * B200 (sm_100a).
 *
 * Conventions for every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller unless the
 *     field says "host".  The library never frees or retains caller memory.
 *   - Calls are asynchronous on the CUDA stream passed as `void *stream`
 *     (a cudaStream_t; NULL = default stream).  The library never
 *     synchronises the stream or the device.
 *   - Calls whose data pointers are all device pointers (pvlm_verify_attn,
 *     pvlm_uvprune_select_gather, pvlm_uvprune_similarity, pvlm_spec_accept,
 *     pvlm_acceptance_rate, and pvlm_verify_step without host buffers) allocate
 *     nothing and read nothing back, so they may be issued on a stream that is
 *     being captured into a CUDA graph; the graph then replays them on the
 *     same buffers.  pvlm_parallel_decode and pvlm_verify_step with host
 *     buffers read results on the host and cannot be captured.
 *   - Scratch memory is caller-provided: `workspace` must hold at least the
 *     number of bytes the matching *_workspace_bytes query returns for the
 *     same parameter struct, and be 256-byte aligned.  Workspace contents are
 *     undefined before and after a call.  Two calls that may overlap on the
 *     GPU need distinct workspaces.
 *   - Outputs are overwritten, never accumulated; inputs are never modified.
 *   - Argument errors are detected on the host before anything is launched
 *     and reported through the return value; no device-side trap exists.
 *   - Results are run-to-run deterministic (no floating-point atomics).
 *   - bf16 tensors are passed as `void *` (2 bytes per element).
 *   - All base pointers of bf16 / fp32 tensors must be 16-byte aligned and
 *     bf16 strides must be multiples of 8 elements.
 */
#ifndef PVLM_H
#define PVLM_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int pvlm_status;
enum {
  PVLM_OK = 0,
  PVLM_ERR_INVALID_ARG = 1, /* NULL where data is required, negative size, bad stride or alignment */
  PVLM_ERR_UNSUPPORTED = 2, /* shape outside the compiled set (see each call) */
  PVLM_ERR_WORKSPACE = 3,   /* workspace NULL, misaligned or too small */
  PVLM_ERR_CUDA = 4,        /* a launch failed; see pvlm_last_cuda_error() */
  PVLM_ERR_TOO_LARGE = 5,   /* size beyond the fixed capacity of a no-allocation entry point */
  PVLM_ERR_TIMEOUT = 6      /* a bounded on-device wait expired; outputs of that call are undefined */
};

/* Human-readable name of a status code (static storage). */
const char *pvlm_status_string(pvlm_status s);
/* cudaError_t (as int) of the most recent failed launch on this host thread, 0 if none. */
int pvlm_last_cuda_error(void);
/* Library version: major * 1000 + minor. */
int pvlm_version(void);

/* Process-wide switches for tests and A/B measurements; none selects a CPU path and none is needed for
 * normal use.  Their defaults are read ONCE from the environment (the variable named beside each), so the
 * launch path of every call is free of environment lookups; afterwards only this function changes them.
 * It returns the previous value, or -1 for an unknown option or a negative value.  A change takes effect
 * for calls (and workspace queries) issued after it returns; do not change a switch between a workspace
 * query and the call it sizes. */
enum {
  PVLM_OPT_ATTN_MMA_SYNC = 0,  /* 1: pvlm_verify_attn runs its first implementation (mma.sync kernels) instead of
                                  the tcgen05 one: a second implementation for tests.  PVLM_ATTN_IMPL=mma      */
  PVLM_OPT_SELECT_ONE_CTA = 1, /* 1: the Top-K selection runs its single-CTA kernels instead of the 8-CTA cluster
                                  kernel: a second implementation for tests.  PVLM_SELECT_IMPL=cta             */
  PVLM_OPT_ATTN_MAX_CTAS = 2,  /* n > 0: the tcgen05 attention uses at most n persistent CTAs, so that small test
                                  shapes exercise long tile runs and many segments per CTA.  PVLM_TC_CTAS=n    */
  PVLM_OPT_COUNT = 3
};
int pvlm_set_option(int option, int value);

/* ------------------------------------------------------------------------
 * Window-verify grouped-query attention with attention-mass emission.
 *
 * The target model verifies the gamma drafted tokens in one parallel pass
 * over the full multimodal context (paper Sec. 2.2; Sec. 4.2, Stage II).
 * Per layer: window row r (0 <= r < R, R = gamma + 1) of query head h attends
 * keys j in [0, n_ctx + r] of KV head floor(h / (Hq / Hkv)):
 *     s_j = softmax_scale * <q[r,h,:], k[j,g,:]>,  P = softmax_j(s),
 *     o[r,h,:] = sum_j P_j v[j,g,:],  lse[h,r] = log sum_j exp(s_j).
 * The attention mass of key j is sum over all h and r of P_j: the
 * attention-score signal that attention-guided pruning ranks visual tokens
 * by (paper Sec. 3, Challenge 2), which a block-wise attention kernel does
 * not otherwise expose.
 *
 * T = n_ctx + R rows of k and v are read per layer: the committed context
 * followed by the window's own rows.  n_layers > 1 batches independent
 * layers into one launch.
 *
 * Supported: D in {64, 128}; Hq % Hkv == 0; 1 <= R; (Hq / Hkv) * R <= 128;
 * n_ctx >= 0; n_layers >= 1.  Anything else returns PVLM_ERR_UNSUPPORTED.
 * bf16 inputs, fp32 accumulation; o is rounded to bf16 once at the end.
 * ---------------------------------------------------------------------- */
typedef struct {
  const void *q;        /* bf16 [n_layers][R][Hq][D], layer stride q_layer_stride            */
  const void *k;        /* bf16 [n_layers][T][Hkv][D], strides below                          */
  const void *v;        /* bf16, same layout and strides as k                                  */
  void *o;              /* bf16 [n_layers][R][Hq][D], same layer stride as q                   */
  float *lse;           /* fp32 [n_layers][Hq][R] natural-log lse; nullable                    */
  float *mass;          /* fp32 [n_mass][T], row stride mass_layer_stride; nullable => the
                           mass pass is skipped for the whole call.  n_mass = n_mass_layers
                           if mass_layers is given, else n_layers                              */
  const int *mass_layers; /* HOST array [n_mass_layers] of layer indices (each in
                           [0, n_layers)) whose mass is wanted, row i of `mass` receiving
                           layer mass_layers[i]; NULL => every layer.  At most 8 entries.
                           The variation score needs only its two end layers (Eq. 2).          */
  int n_mass_layers;
  int n_layers, R, Hq, Hkv, D, n_ctx;
  long long q_layer_stride;    /* elements */
  long long kv_layer_stride;   /* elements */
  long long kv_token_stride;   /* elements, >= D (token-major [T][Hkv][D] and head-major      */
  long long kv_head_stride;    /* elements, >= D  [Hkv][T][D] caches are both expressible)     */
  long long mass_layer_stride; /* elements, >= T                                               */
  float softmax_scale;         /* 0 => 1/sqrt(D)                                               */
  void *workspace;
  size_t workspace_bytes;
  void *prof_event_begin; /* optional cudaEvent_t pair (NULL = off): recorded on the stream right before   */
  void *prof_event_end;   /* and right after the one kernel that streams K and V, for per-kernel timing   */
  int max_ctas;           /* 0 = one persistent CTA per SM.  A smaller value leaves SMs free for kernels   */
                          /* of another stream (the draft model's decode steps run beside verification:   */
                          /* paper Sec. 4.2, Stage II); the workspace query must see the same value.      */
} pvlm_attn_params;

/* Host-only; needs no GPU.  Returns 0 if the parameters are unsupported. */
size_t pvlm_verify_attn_workspace_bytes(const pvlm_attn_params *p);
pvlm_status pvlm_verify_attn(const pvlm_attn_params *p, void *stream);
/* Health check of the last pvlm_verify_attn issued with this parameter block (same workspace):
 * every wait inside the kernels is bounded, and one that expires records it in the workspace
 * instead of hanging.  This call SYNCHRONISES `stream`, reads that word and returns PVLM_OK or
 * PVLM_ERR_TIMEOUT.  Optional: results of a call that timed out are undefined either way.
 * (The word is cleared by the call's first kernel, so it always describes the last call.) */
pvlm_status pvlm_verify_attn_check(const pvlm_attn_params *p, void *stream);

/* ------------------------------------------------------------------------
 * UV-Prune: debiased score, Top-K selection, gather into the draft cache.
 *
 * score_i = mass_cur[vis_start + i] - mass_ref[vis_start + i] for the m
 * visual tokens: the layer-to-layer variation of the relevance signal summed
 * over layers (paper Eq. 2), which telescopes to the difference of its two
 * end layers and cancels the layer-invariant positional part (Appendix E).
 * One fp32 subtraction, round to nearest.  mass_ref == NULL ranks by the raw
 * signal.  The k largest scores are kept (Eq. 3; k = (1 - alpha) m, Eq. 5);
 * equal scores are kept lower index first (-0.0 == +0.0; NaN ranks below
 * every number); kept_idx is ascending, relative to vis_start.
 *
 * If src_k is non-NULL the kept rows are gathered, per layer and for K and V:
 *   dst = [ src[0, vis_start) ; src[vis_start + kept_idx[.]] ; src[vis_start + m, src_len) ]
 * i.e. the draft context keeps the selected visual tokens and everything
 * else (paper Sec. 4.2, Stage I: draft prefix = (V*, X_{1:n})).  Byte copy.
 *
 * Supported: 0 <= k <= m <= 2^24; row_bytes % 16 == 0; src/dst 16-byte aligned.
 * ---------------------------------------------------------------------- */
typedef struct {
  const float *mass_cur; /* fp32 [>= vis_start + m]                                           */
  const float *mass_ref; /* fp32 [>= vis_start + m]; nullable                                 */
  int vis_start, m, k;
  int *kept_idx;         /* int32 [k] out                                                      */
  float *score;          /* fp32 [m] out; nullable                                             */
  const void *src_k, *src_v; /* [n_layers][src_len][row_bytes]; both NULL => select only      */
  void *dst_k, *dst_v;       /* [n_layers][src_len - m + k][row_bytes]; may be NULL if that is 0 rows */
  int n_layers, src_len;
  long long row_bytes;
  long long src_layer_stride_bytes, dst_layer_stride_bytes;
  void *workspace;
  size_t workspace_bytes;
} pvlm_prune_params;

size_t pvlm_uvprune_workspace_bytes(const pvlm_prune_params *p);
pvlm_status pvlm_uvprune_select_gather(const pvlm_prune_params *p, void *stream);

/* ------------------------------------------------------------------------
 * Vision-text similarity signal of UV-Prune on token representations.
 *
 * The paper's own pruning criterion (Sec. 4.1): the cosine similarity
 * S_ij = V_i.X_j / (|V_i||X_j|) between visual token i and text token j in
 * one early layer of the target (Eq. 1), summed over the text tokens
 * (the inner sum of Eq. 2):  sim[i] = sum_j S_ij,  i = 0..m-1.
 * Calling it for the last and for the first layer of the early-layer set and
 * passing the two results as mass_cur / mass_ref of
 * pvlm_uvprune_select_gather gives Eq. 2 (which telescopes to the difference
 * of its two end layers), Eq. 3 and the gather.  A zero vector has similarity
 * 0 with everything.  fp32 accumulation.
 *
 * hidden: bf16 [rows][d] token representations of one layer, row stride
 * hidden_row_stride elements; visual rows [vis_start, vis_start+m), text
 * rows [text_start, text_start+n).
 * n_layers > 1 computes that many layers in one call (the two end layers of
 * Eq. 2 normally): layer l's hidden states start hidden_layer_stride elements
 * after layer l-1's and its result goes to sim + l * sim_layer_stride; each
 * kernel then covers all layers in one launch.  n_layers <= 1 is one layer
 * and the two layer strides are ignored.
 * Supported: d % 8 == 0, 8 <= d <= 16384; hidden 16-byte aligned, row and
 * layer strides multiples of 8; m >= 0, n >= 0; n_layers <= 65535.
 * ---------------------------------------------------------------------- */
typedef struct {
  const void *hidden;
  long long hidden_row_stride;
  int vis_start, m, text_start, n, d;
  float *sim;             /* fp32 [m] out ([n_layers][sim_layer_stride] with several layers) */
  void *workspace;
  size_t workspace_bytes;
  int n_layers;                   /* 0 or 1: one layer */
  long long hidden_layer_stride;  /* elements, used when n_layers > 1 */
  long long sim_layer_stride;     /* elements, >= m, used when n_layers > 1 */
} pvlm_similarity_params;

size_t pvlm_uvprune_similarity_workspace_bytes(const pvlm_similarity_params *p);
pvlm_status pvlm_uvprune_similarity(const pvlm_similarity_params *p, void *stream);

/* ------------------------------------------------------------------------
 * Vocab softmax + lossless accept / reject + residual resampling.
 *
 * p_t = softmax(target_logits[t] / temperature), t = 0..gamma;
 * q_t = softmax(draft_logits[t] / temperature), t = 0..gamma-1.
 * Drafted token x_t is accepted with probability min{1, p_t(x_t)/q_t(x_t)}
 * (paper Sec. 2.2), evaluated as u_t * q_t(x_t) < p_t(x_t) in fp32; at the
 * first rejection n a replacement is drawn from norm(max(0, p_n - q_n))
 * (same section); if all gamma are accepted one token is drawn from
 * p_gamma.  The draw is an inverse CDF in vocabulary order with uniform
 * u_gamma: the smallest j whose cumulative weight exceeds u * total.
 *
 * `batch` independent sequences share gamma and V; sequence b uses
 * target_logits + b * target_batch_stride, etc. (a batch stride of 0 lets
 * every sequence read the same logits); small per-sequence arrays are densely
 * packed [batch][...].  Full-probability outputs, if requested, use the same
 * strides as the logits (so they need non-zero batch strides).
 *
 * gamma = 0 is plain sampling: nothing is verified, one token is drawn from
 * p_0 with uniform u_0 (the draft model's own decoding step uses the call
 * this way on its logits); draft_logits and draft_tokens may then be NULL.
 *
 * Supported: 0 <= gamma <= 64; 1 <= V < 2^31; 1 <= batch <= 65535.  Rows are
 * read with 16-byte loads when the logit base pointers are 16-byte aligned
 * and all logit strides are multiples of 4 elements, else element by element.
 *
 * One kernel launch.  Inside it a few thread blocks wait (for microseconds)
 * for the block that determines n_accept; that wait is bounded to one second,
 * and if it ever expired the drawn token would be missing:
 * out_tokens[n_accept] == -1 is the mark of that failure.
 * ---------------------------------------------------------------------- */
typedef struct {
  const float *target_logits;  /* fp32 [batch][gamma+1][V]                                    */
  const float *draft_logits;   /* fp32 [batch][gamma][V]                                      */
  long long target_row_stride, draft_row_stride;     /* elements                               */
  long long target_batch_stride, draft_batch_stride; /* elements                               */
  const int *draft_tokens;     /* int32 [batch][gamma], each in [0, V)                         */
  const float *uniforms;       /* fp32 [batch][gamma+1] in [0,1): gamma accept tests, 1 draw   */
  int batch, gamma, V;
  float temperature;           /* 0 or 1 => 1                                                  */
  int *n_accept;               /* int32 [batch] out, in [0, gamma]                             */
  int *out_tokens;             /* int32 [batch][gamma+1] out: n_accept drafts, the drawn token, then -1 */
  float *p_tok, *q_tok;        /* fp32 [batch][gamma] out: p_t(x_t), q_t(x_t) for every t; nullable     */
  float *lse_p, *lse_q;        /* fp32 [batch][gamma+1], [batch][gamma] out (of logits/temperature); nullable */
  float *probs_p, *probs_q;    /* fp32 full probabilities, same strides as the logits; nullable (tests) */
  void *workspace;
  size_t workspace_bytes;
} pvlm_accept_params;

size_t pvlm_spec_accept_workspace_bytes(const pvlm_accept_params *p);
pvlm_status pvlm_spec_accept(const pvlm_accept_params *p, void *stream);

/* ------------------------------------------------------------------------
 * The two decisions of the step on their own, from given scores / probabilities.
 *
 * Kept indices and accepted lengths are integer results of floating-point
 * inputs.  These two calls take those inputs from the caller instead of
 * computing them, so that a test can feed values computed elsewhere (e.g. by an
 * independent CPU implementation) and compare the integer results bit for bit.
 * They run the same device code as the full calls.
 *
 * pvlm_select_from_scores: Top-K of paper Eq. 3 over given scores.
 *   score fp32 [m] (device); kept_idx int32 [k] out, ascending; the k largest
 *   scores, equal scores lower index first, -0.0 == +0.0, NaN below every
 *   number: pvlm_uvprune_select_gather with mass_cur = score, mass_ref = NULL,
 *   vis_start = 0 and no gather.  Workspace as pvlm_uvprune_workspace_bytes
 *   reports for the same m.  Errors as for that call.
 *
 * pvlm_accept_from_probs: the accept rule of paper Sec. 2.2 over given token
 *   probabilities.  p_tok, q_tok fp32 [batch][gamma] (device): p_t(x_t) and
 *   q_t(x_t) of the drafted tokens; uniforms fp32 [batch][uniform_stride]
 *   (device), the first gamma of each row used (uniform_stride >= gamma; pass
 *   gamma + 1 for the array pvlm_spec_accept takes); n_accept int32 [batch]
 *   out: the first t with not (u_t * q_t < p_t), evaluated as in
 *   pvlm_spec_accept (one rounded fp32 multiply, strict compare), or gamma if
 *   there is none.  0 <= gamma, 1 <= batch.  No workspace.
 * ---------------------------------------------------------------------- */
pvlm_status pvlm_select_from_scores(const float *score, int m, int k, int *kept_idx, void *workspace,
                                    size_t workspace_bytes, void *stream);
pvlm_status pvlm_accept_from_probs(const float *p_tok, const float *q_tok, const float *uniforms, int uniform_stride,
                                   int gamma, int batch, int *n_accept, void *stream);

/* ------------------------------------------------------------------------
 * One whole verify -> prune -> accept step from HOST-side step inputs.
 *
 * The verification round of the parallel decoding pipeline (paper Sec. 4.2,
 * Stage II; Appendix B) as one call: copy this step's inputs from host memory
 * into caller-provided device buffers, run the three stages in order on
 * `stream`, copy the step's results back.  The KV cache of the committed
 * context is resident device state (like weights) and is not copied; only the
 * window's own K/V rows are written into it at token rows [n_ctx, n_ctx + R).
 *
 * `attn`, `prune`, `accept` are complete parameter blocks as for the three
 * calls above (all their pointers are device pointers; prune.mass_cur /
 * mass_ref normally point at rows of attn.mass).  A stage whose `run_*` flag
 * is 0 is skipped.  Every h_* pointer is a HOST pointer (pinned memory makes
 * the copies asynchronous) and may be NULL, which skips that copy:
 *   h_q            bf16 [n_layers][R][Hq][D]        -> attn.q
 *   h_k_window/v   bf16 [n_layers][R][Hkv][D]       -> attn.k / attn.v rows n_ctx.. of a token-major cache
 *                                                      (kv_head_stride == D, kv_token_stride == Hkv*D), or
 *                  bf16 [n_layers][Hkv][R][D]       -> the same rows of a head-major cache (kv_token_stride
 *                                                      == D, kv_layer_stride == Hkv*kv_head_stride);
 *                                                      other stride combinations: PVLM_ERR_UNSUPPORTED
 *   h_target_logits fp32 [batch][gamma+1][V] dense  -> accept.target_logits (dense strides required)
 *   h_draft_logits  fp32 [batch][gamma][V] dense    -> accept.draft_logits
 *   h_draft_tokens, h_uniforms                      -> accept.draft_tokens, accept.uniforms
 *   h_o            <- attn.o;  h_n_accept, h_out_tokens <- accept;  h_kept_idx <- prune.kept_idx
 * The call returns after enqueueing; results in host memory are valid once
 * the stream has been synchronised by the caller.
 * ---------------------------------------------------------------------- */
typedef struct {
  pvlm_attn_params attn;
  pvlm_prune_params prune;
  pvlm_accept_params accept;
  int run_attn, run_prune, run_accept;
  const void *h_q, *h_k_window, *h_v_window;
  const float *h_target_logits, *h_draft_logits;
  const int *h_draft_tokens;
  const float *h_uniforms;
  void *h_o;
  int *h_n_accept, *h_out_tokens, *h_kept_idx;
  /* Optional overlap (all three NULL = everything on `stream`): a second cudaStream_t and two cudaEvent_t
   * owned by the caller.  The accept inputs (logits, drafts, uniforms) are then uploaded on copy_stream
   * while the attention runs, the accept stage itself (which depends on nothing else in the step) runs on
   * copy_stream behind them, and o is downloaded on copy_stream while select/gather run.  The call still
   * orders everything so that synchronising `stream` alone is enough afterwards. */
  void *copy_stream, *event_a, *event_b;
  /* Optional HOST int32 [1] (NULL = off): receives the status word of the attention stage (of the last attention call
   * on attn.workspace if run_attn is 0) with the other results: 0 = fine, non-zero = a bounded wait inside its kernels
   * expired and o, mass and everything computed from them (kept_idx, the gathered cache) are undefined for this step.
   * Without it, call pvlm_verify_attn_check(&attn, stream) after the stream has been synchronised to learn the same. */
  int *h_attn_status;
} pvlm_step_params;

pvlm_status pvlm_verify_step(const pvlm_step_params *p, void *stream);

/* ------------------------------------------------------------------------
 * Token-wise acceptance rate of a given text (the paper's metric A).
 *
 * Appendix "Tasks and Metrics": the text a pruned model wrote is scored by
 * token-wise speculative sampling under the full-context target: token x_n,
 * whose writer had distribution q_n, counts as accepted iff
 * u_n < p_n(x_n) / q_n(x_n) (evaluated as u_n * q32 < p32 in fp32, like
 * pvlm_spec_accept), every position on its own, and A = accepted / N.
 * One pass over the 2N logit rows (8 N V bytes): the bandwidth-bound form of
 * the vocab softmax.
 *
 * All pointers are DEVICE pointers.  accepted / p_tok / q_tok hold one value
 * per token; *n_accepted receives the count (the call zeroes it first).
 * Tokens outside [0, V) count as rejected with p = 0, q = 1.  N = 0 is a
 * no-op that writes *n_accepted = 0.  Supported: 0 <= N < 2^30, 1 <= V < 2^31.
 * ---------------------------------------------------------------------- */
typedef struct {
  const float *target_logits, *draft_logits;   /* fp32 [N][row stride], first V of a row used */
  long long target_row_stride, draft_row_stride;
  const int *tokens;                           /* int32 [N]                                   */
  const float *uniforms;                       /* fp32 [N] in [0,1)                           */
  int N, V;
  float temperature;                           /* 0 or 1 => 1                                 */
  int *accepted;                               /* int32 [N] out: 1 / 0                        */
  float *p_tok, *q_tok;                        /* fp32 [N] out, nullable                      */
  int *n_accepted;                             /* int32 [1] out                               */
  void *workspace;
  size_t workspace_bytes;
} pvlm_rate_params;

size_t pvlm_acceptance_rate_workspace_bytes(const pvlm_rate_params *p);
pvlm_status pvlm_acceptance_rate(const pvlm_rate_params *p, void *stream);

/* ------------------------------------------------------------------------
 * Parallel decoding: the Pre-verify / Post-verify round loop on two streams.
 *
 * Stage II of the paper (Sec. 4.2 "Parallel Decoding"; Algorithm 1 and the
 * appendix "Parallel Pipeline Details"): in every round the target verifies
 * while the draft model writes `gamma` further tokens, each on its own
 * stream; a rejection commits the replacement token, drops every other draft
 * (the draft cache rolls back to the committed prefix) and returns to
 * Pre-verify.
 *   Pre-verify round : the draft writes d_0..d_{gamma-1}; d_0 alone is tested.
 *                      accepted -> d_0 committed, gamma-1 drafts stay pending,
 *                      next round is Post-verify; rejected -> replacement
 *                      committed, drafts dropped.
 *   Post-verify round: all pending drafts are tested in one batch while the
 *                      draft writes gamma more behind them.  All accepted ->
 *                      committed, the new gamma drafts become pending (no
 *                      bonus token); else accepted prefix + replacement
 *                      committed, everything else dropped, next is Pre-verify.
 * The two models are stood in for by logit tables: row i of target_logits /
 * draft_logits is that model's distribution for generated position i.  Each
 * round runs, on `draft_stream`, the gamma draws from the draft rows
 * (pvlm_spec_accept with gamma = 0, batch = gamma) and, on `target_stream`,
 * the accept / reject / resample kernels over the tokens under test; if
 * target_attn / draft_attn are given, the round also runs the two models'
 * attention over their caches as they stand in that round (the outputs are not
 * used; the logit tables stand in for the rest of the forward):
 *   target: one call with n_ctx = target_attn->n_ctx + (tokens committed so
 *           far) and R = (tokens under test) + 1: the committed tokens have
 *           become context, the window holds the last committed token and the
 *           drafts being verified;
 *   draft : gamma calls (R = 1), step t with n_ctx = draft_attn->n_ctx +
 *           (tokens committed) + (drafts pending) + t: the draft's cache grows
 *           by one row per token it writes, and after a rejection it is
 *           truncated to the committed prefix (the replacement token is the
 *           next step's input), so the next round starts from there.
 * The blocks' n_ctx are the context lengths before the first generated token;
 * their k / v must hold n_ctx + K + 2 * gamma + 1 token rows and their
 * workspaces must cover every round's shape (sizing them with n_ctx + K +
 * 2 * gamma and R = gamma + 1 does; a round whose call does not fit returns
 * PVLM_ERR_WORKSPACE).  A bounded wait that expires inside one of these
 * attention calls ends the loop with PVLM_ERR_TIMEOUT.  Random numbers are
 * indexed by round: u_draft[r][s] draws the s-th token drafted in round r,
 * u_accept[r][s] tests the s-th token verified in round r, u_resample[r]
 * draws round r's replacement.
 *
 * The call is synchronous: it returns after K tokens have been committed
 * (both streams idle).  tokens, round_log, n_rounds, round_ms are HOST
 * pointers; everything else in the block is a DEVICE pointer.  Errors: bad
 * sizes or NULL pointers PVLM_ERR_INVALID_ARG; P < K + 2*gamma + 1 or
 * max_rounds exhausted PVLM_ERR_TOO_LARGE; workspace as for the other calls.
 * ---------------------------------------------------------------------- */
#define PVLM_DECODE_LOG_COLS 9
typedef struct {
  const float *target_logits, *draft_logits;  /* fp32 [P][row_stride], first V of a row used */
  long long row_stride;                       /* elements, >= V                              */
  int P, V, gamma, K;                         /* 1 <= gamma <= 64; K tokens to generate       */
  float temperature;
  const float *u_draft, *u_accept;            /* fp32 [max_rounds][gamma] in [0,1)            */
  const float *u_resample;                    /* fp32 [max_rounds]                            */
  int max_rounds;                             /* K rounds always suffice                      */
  int *tokens;                                /* HOST int32 [K] out                           */
  int *round_log;                             /* HOST int32 [max_rounds][PVLM_DECODE_LOG_COLS] out, nullable:
                                                 mode (0 Pre, 1 Post), verified, accepted, committed, dropped, start,
                                                 target_ctx, draft_ctx, draft_keep: generated tokens in the verification
                                                 call's context, in the draft's cache before the round's first draft step,
                                                 and in the draft's cache after the round's commit or rollback          */
  int *n_rounds;                              /* HOST int32 out, nullable                     */
  float *round_ms;                            /* HOST fp32 [max_rounds] out, nullable: device time of each round  */
  const pvlm_attn_params *target_attn;        /* HOST pointer to a complete block, nullable   */
  const pvlm_attn_params *draft_attn;         /* HOST pointer to a complete block, nullable   */
  int serial;                                 /* 1 = vanilla SD order for comparison: the draft's work, then the
                                                 target's, on target_stream only (same tokens)                */
  void *workspace;
  size_t workspace_bytes;
} pvlm_decode_params;

size_t pvlm_parallel_decode_workspace_bytes(const pvlm_decode_params *p);
pvlm_status pvlm_parallel_decode(const pvlm_decode_params *p, void *target_stream, void *draft_stream);

/* ------------------------------------------------------------------------
 * Draft window size from measured forward times (host arithmetic, no GPU).
 *
 * The window equals the pruned speed ratio c* = T_p / T_q(alpha) (paper
 * Eq. 6).  c* is rarely an integer; the paper calls rounding down the wiser
 * choice when the window is aggressive relative to the mean accepted length
 * and rounding up the sensible one for narrow windows with high accepted
 * lengths (Appendix A, "Window Size Selection"), and leaves the choice to the
 * user; the five window sizes it uses itself all equal c* rounded to the
 * nearest integer.  mode: 0 = nearest, 1 = down, 2 = up.  Never below 1.
 * Returns 0 if a time is not positive or the mode is unknown.
 * ---------------------------------------------------------------------- */
enum { PVLM_ROUND_NEAREST = 0, PVLM_ROUND_DOWN = 1, PVLM_ROUND_UP = 2 };
int pvlm_window_size(double t_target, double t_draft, int mode);

/* ------------------------------------------------------------------------
 * Top-K selection that needs no caller-side scratch allocation.
 * (The paper has no counterpart: this is a packaging variant of the
 * selection half of pvlm_uvprune_select_gather, for callers that cannot
 * allocate device memory.)
 *
 * Some callers of this library cannot call cudaMalloc at the point where
 * they need a selection: code running inside a pre-sized memory arena whose
 * budget is fixed at start-up, plug-ins loaded into a host process that owns
 * all device memory, or a latency-critical loop where an allocation (which
 * may synchronise the device) is not acceptable.  pvlm_uvprune_select_gather
 * asks such a caller for a workspace it has no way to provide.  This entry
 * point computes exactly the same kept_idx (same score, same tie rule, same
 * ascending order) but keeps its scratch (one 32-bit key per visual token) in
 * a fixed array inside the library's device image.
 *
 * Capacity: m <= PVLM_SELECT_STATIC_MAX_M.  A larger m returns
 * PVLM_ERR_TOO_LARGE and launches nothing.  The array costs
 * 4 * PVLM_SELECT_STATIC_MAX_M bytes (1 MiB) of device memory on every GPU
 * that loads the library, from load until process exit.
 *
 * The call allocates nothing and frees nothing, on host or device.  The first
 * call on each device looks up the array's device address (a driver query, no
 * allocation); make that first call outside any CUDA stream capture.
 *
 * All calls on one device share the one array.  Nothing in it has to start at
 * zero: every call overwrites the first m keys before reading them, so what
 * an earlier call left behind is never observed.  Two calls that may run on
 * the GPU at the same time (different streams without an ordering between
 * them) race on the array and give undefined kept_idx; order them on one
 * stream or with events.
 *
 * mass_cur, mass_ref, vis_start, m, k, kept_idx, score: as in pvlm_prune_params
 * (mass_ref and score nullable).  No gather is performed.
 * ---------------------------------------------------------------------- */
#define PVLM_SELECT_STATIC_MAX_M 262144
pvlm_status pvlm_uvprune_select_static(const float *mass_cur, const float *mass_ref, int vis_start, int m, int k,
                                       int *kept_idx, float *score, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PVLM_H */
