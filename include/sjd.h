/*
 * libsjd - one Speculative Jacobi Decoding (SJD) iteration on one GPU (sm_100a).
 *
 * The library runs the per-iteration hot path of SJD for a decoder-only
 * image-token transformer (arXiv 2410.01699, Sec. 4.1 Steps 1-4, Eqs. 1-3,
 * Sec. 4.2): a window of W draft tokens goes through the model in a single
 * forward pass against a KV cache, each draft is accepted with probability
 * min(1, p/q), the first rejected position is resampled from
 * norm(max(0, p - q)), the rest of the window is re-drawn from the new
 * distributions, and the window slides over the accepted tokens.
 *
 * Conventions
 *   - Every function returns SJD_OK (0) or a negative sjd_status.  Nothing
 *     throws, aborts or prints.
 *   - "device" pointers are CUDA device pointers of the current device;
 *     "host" pointers are ordinary host memory.  Pointers named in
 *     sjd_step_out may be device memory or pinned (mapped) host memory.
 *   - The caller owns all device memory: weights, the workspace and the
 *     outputs.  The library owns only the small host-side context.  Weights
 *     are borrowed for the lifetime of the context and never written.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default
 *     stream).  Work is enqueued asynchronously; no call synchronises the
 *     device except sjd_init (table upload) and sjd_last_device_status.
 *   - Matrices are row-major [out_features][in_features] (y = x W^T).
 *   - All sequences of a batch share n_generate and the sampling configuration (prompt lengths may
 *     differ: sjd_prefill_ragged); the Philox counter carries the sequence id.
 *
 * Random numbers: Philox4x32-10 (Salmon et al., SC'11), key = 64-bit seed,
 * counter = (absolute position, step index, sequence id, stream tag).
 * Stream tag 0: word 0 -> acceptance test (Eq. 1), word 1 -> residual
 * resample (Eq. 2), word 2 -> re-draft (Eq. 3).  Stream tag 1: word 0 ->
 * random token of a freshly initialised slot, floor(word * V / 2^32).  A
 * uniform is (word >> 8) * 2^-24.  The first window uses step 0xFFFFFFFF.
 */
#ifndef SJD_H_
#define SJD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sjd_ctx sjd_ctx; /* opaque; created by sjd_init, freed by sjd_destroy */

typedef enum {
  SJD_OK = 0,
  SJD_ERR_BAD_ARG = -1,        /* null pointer, non-positive size, T <= 0, top_k < 1 ...      */
  SJD_ERR_CAPACITY = -2,       /* batch/window/sequence/workspace/vocab beyond what was sized */
  SJD_ERR_UNSUPPORTED = -3,    /* shape or dtype the kernels do not cover                     */
  SJD_ERR_CUDA = -4,           /* a CUDA runtime call failed; see sjd_last_cuda_error         */
  SJD_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait ran out                          */
  SJD_ERR_STATE = -6           /* call out of order (step before prefill ...)                 */
} sjd_status;

typedef enum { SJD_F32 = 0, SJD_BF16 = 1 } sjd_dtype;

/* How new window slots are initialised (Sec. 4.2). */
typedef enum {
  SJD_INIT_RANDOM = 0,     /* uniform random token; carries q = 1/V                         */
  SJD_INIT_COPY_ABOVE = 1, /* token at position - grid_stride (strategy (b)); q = point mass */
  SJD_INIT_COPY_LEFT = 2,  /* token at position - 1 (strategy (a)); q = point mass           */
  SJD_INIT_RESAMPLE_LEFT = 3, /* strategy (c): drawn from the distribution predicted at the left neighbour, */
                           /* i.e. from the most recent logits row of the nearest position to the left   */
                           /* that has been through a pass (row min(t - 1 - n, W_eff - 1) of this pass);  */
                           /* q = that row's top-k softmax; first window: uniform random token            */
  SJD_INIT_RESAMPLE_ABOVE = 4 /* strategy (d): drawn from the distribution predicted at position -        */
                           /* grid_stride, i.e. from the most recent logits row of that position, which   */
                           /* the context retains in a ring of cfg.max_ring rows (the rows as the         */
                           /* verification saw them: mixed under guidance); no such row (first image      */
                           /* row): uniform random token                                                   */
} sjd_init_kind;

/* Which decoding schedule a step runs: the paper's method, or one of the baselines it is compared with
 * (Table 1 rows A-D: plain next-token sampling is SJD with window 1; Sec. 3.2; the no-refinement ablation). */
typedef enum {
  SJD_SCHEDULE_SJD = 0,       /* Sec. 4.1: accept with min(1, p/q), resample the first rejection, re-draft the rest */
  SJD_SCHEDULE_JACOBI = 1,    /* Sec. 3.2: every slot re-drawn from this pass's row with the uniform of its      */
                              /* position (re-draft word, step index 0); the unchanged prefix and the first    */
                              /* changed slot are fixed; no q is used                                            */
  SJD_SCHEDULE_NO_REFINE = 2  /* Eqs. 1-2 only: the slots after the first rejection are re-initialised (Sec. 4.2) */
                              /* instead of re-drawn by Eq. 3                                                     */
} sjd_schedule_kind;

/* The law a draft token was drawn from (Step 1: "the probability corresponding to the draft"). */
typedef enum {
  SJD_Q_ROW = 0,     /* top-k softmax of the logits row that produced it one iteration ago */
  SJD_Q_UNIFORM = 1, /* 1/V                                                                */
  SJD_Q_ONEHOT = 2,  /* point mass on the draft itself                                     */
  SJD_Q_RING = 3     /* top-k softmax of a retained logits row (SJD_INIT_RESAMPLE_ABOVE)   */
} sjd_q_kind;

/* bits of sjd_step_out.flags */
#define SJD_FLAG_NEAR_TIE_ACCEPT 1u /* some scanned row had |u - min(1,p/q)| < 1e-4 with p/q < 1  */
#define SJD_FLAG_RESIDUAL_EMPTY 4u  /* sum max(0,p-q) == 0 at the rejected row: sampled from p    */
#define SJD_FLAG_NONFINITE 8u       /* a logits row held NaN or +inf (treated as -inf)            */
#define SJD_FLAG_DONE 16u           /* all n_generate tokens of this sequence are fixed           */

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, ffn_hidden, vocab;
  float rope_theta; /* rotary base; pairs (i, i + head_dim/2), angle pos * theta^(-2i/head_dim) */
  float rms_eps;
  int32_t dtype;    /* sjd_dtype of weights, activations, KV cache and stored logits */
  int32_t max_batch, max_seq, max_window;
  int32_t max_ring; /* logits rows retained per image for SJD_INIT_RESAMPLE_ABOVE: at least grid_stride +   */
                    /* window (each costs vocab elements of dtype in the workspace); 0 if that strategy is  */
                    /* not used                                                                            */
  int32_t kv_pages; /* 0: every sequence owns max_seq cache rows.  > 0: paged cache (the paper has none; a    */
                    /* serving-side layout): the batch shares a pool of kv_pages pages of SJD_KV_PAGE         */
                    /* positions, and sjd_prefill gives each sequence the ceil((prompt_len + n_generate) /    */
                    /* SJD_KV_PAGE) pages it needs (SJD_ERR_CAPACITY when the pool is too small); results are */
                    /* identical to the contiguous layout                                                     */
} sjd_model_cfg;
#define SJD_KV_PAGE 64

/* Device pointers, borrowed.  Per-layer entries are HOST arrays of n_layers device pointers. */
typedef struct {
  const void *tok_emb;    /* [vocab][d_model]                 */
  const void *final_norm; /* [d_model]                        */
  const void *lm_head;    /* [vocab][d_model]                 */
  const void *const *attn_norm; /* [d_model]                  */
  const void *const *wq;        /* [n_heads*head_dim][d_model]    */
  const void *const *wk;        /* [n_kv_heads*head_dim][d_model] */
  const void *const *wv;        /* [n_kv_heads*head_dim][d_model] */
  const void *const *wo;        /* [d_model][n_heads*head_dim]    */
  const void *const *ffn_norm;  /* [d_model]                  */
  const void *const *w_gate;    /* [ffn_hidden][d_model]      */
  const void *const *w_up;      /* [ffn_hidden][d_model]      */
  const void *const *w_down;    /* [d_model][ffn_hidden]      */
  /* QK-norm variant (the Chameleon family of Sec. 5.1): per-layer gains [head_dim]; every head of q and of k  */
  /* is RMS-normalised over its head_dim entries (eps = rms_eps) and multiplied by the gain before the rotary */
  /* step.  Both NULL: the plain model.                                                                        */
  const void *const *q_norm;
  const void *const *k_norm;
} sjd_weights;

typedef struct {
  float temperature;   /* > 0; logits are divided by it before top-k (the paper has none: 1.0) */
  int32_t top_k;       /* >= 1; entries equal to the k-th largest are all kept; >= V: no filter */
  uint64_t seed;       /* Philox key                                                            */
  int32_t window;      /* W, Jacobi window size (Sec. 4.1)                                      */
  int32_t init;        /* sjd_init_kind                                                         */
  int32_t grid_stride; /* tokens per image row incl. any row-end token (COPY_ABOVE)             */
  int32_t n_generate;  /* N, image tokens to generate per sequence                              */
  int32_t seq_base;    /* global id of sequence 0 of this batch (Philox counter word 2): a batch    */
                       /* sharded over several GPUs draws the same numbers wherever a sequence runs  */
  float guidance;      /* classifier-free guidance weight w (Sec. 5.1 uses 3.0); 0 = no guidance.   */
                       /* With w != 0 the batch holds two streams per image: sequence 2i is image   */
                       /* i's conditional stream, 2i+1 its unconditional one (prompts of one length, */
                       /* different tokens); both share drafts, uniforms and decisions.  Each        */
                       /* stream's logits are stored in cfg.dtype; verification reads every row as   */
                       /* l_u + w (l_c - l_u), evaluated in fp32 as fma(w, l_c - l_u, l_u) and       */
                       /* rounded to cfg.dtype.  Outputs then have batch / 2 entries (one per image)  */
                       /* and the Philox sequence id is seq_base + i.  sjd_verify(_static): must be 0 */
  int32_t schedule;    /* sjd_schedule_kind; 0 = the paper's method                                  */
} sjd_sample_cfg;

/* Results of one step.  Any pointer may be NULL (that output is skipped). */
typedef struct {
  int32_t *n_accepted;      /* [B]    drafts accepted by Eq. 1 this step (0..W)                    */
  int32_t *n_committed;     /* [B]    tokens fixed this step: accepted (+1 resampled); 0 when done */
  int32_t *committed;       /* [B][W] those tokens, left-aligned, rest -1                          */
  int32_t *draft;           /* [B][W] the next window's draft tokens, rest -1                      */
  int32_t *q_kind;          /* [B][W] sjd_q_kind of each new draft, rest -1                        */
  float *q_draft;           /* [B][W] q(draft) of each new draft under its own law, rest 0         */
  int32_t *total_committed; /* [B]    n after the step (prompt + fixed tokens)                     */
  uint32_t *flags;          /* [B]    SJD_FLAG_* bits raised by this step                          */
} sjd_step_out;

/*
 * Bytes of caller-provided device workspace a context needs: KV cache
 * [layer][batch][k|v][kv_head][max_seq][head_dim], two logits buffers
 * [max_batch][max_window][vocab] (this iteration's p rows are the next
 * iteration's q rows: the buffers swap, nothing is copied), activations, GEMM
 * split-K partials, per-row verification scratch and decoding state.
 * Returns 0 for an invalid configuration.
 */
size_t sjd_workspace_bytes(const sjd_model_cfg *cfg);

/*
 * Create a context (Sec. 3.1: the auto-regressive transformer; Sec. 4.1: its
 * use on a window).  `workspace` is device memory of at least
 * sjd_workspace_bytes(cfg), 256-byte aligned, owned by the caller and must
 * outlive the context.  Uploads the rotary table (synchronous).
 * Errors: BAD_ARG (null / non-positive / odd head_dim / n_heads not a
 * multiple of n_kv_heads), CAPACITY (workspace too small), UNSUPPORTED
 * (head_dim > 256, window > 64, unknown dtype), CUDA.
 */
int sjd_init(sjd_ctx **out, const sjd_model_cfg *cfg, const sjd_weights *weights, void *workspace,
             size_t workspace_bytes);

/*
 * Pre-fill (Sec. 4.1, first sentence): run the model over prompt tokens
 * c[0..P-1) so that their keys/values are cached (the last prompt token is
 * the first input of step 0), then build the first window of W freshly
 * initialised drafts (Sec. 4.2).  prompt: device int32 [batch][prompt_len],
 * prompt_len >= 1.  Resets the step index to 0.
 * Errors: BAD_ARG; CAPACITY (batch > max_batch, window > max_window,
 * prompt_len + n_generate > max_seq); CUDA.
 */
int sjd_prefill(sjd_ctx *ctx, int batch, const int32_t *prompt, int prompt_len,
                const sjd_sample_cfg *sample, void *cuda_stream);

/*
 * sjd_prefill for a ragged batch: sequence b uses the first prompt_lens[b] tokens of row b of `prompt`
 * (device int32 [batch][row_stride]); prompt_lens is a HOST array of `batch` lengths in 1..row_stride.
 * Every sequence keeps its own positions (its image starts right after its own prompt: nothing is padded),
 * generates n_generate tokens and finishes on its own; under guidance the two streams of an image must have
 * prompts of one length.  (Sec. 4.1, first sentence: "after pre-filling the tokens of text prompts";
 * prompts of different lengths in one batch are this library's generalisation.)
 * Errors: as sjd_prefill; CAPACITY is judged by the longest prompt.
 */
int sjd_prefill_ragged(sjd_ctx *ctx, int batch, const int32_t *prompt, const int32_t *prompt_lens, int row_stride,
                       const sjd_sample_cfg *sample, void *cuda_stream);

/*
 * One SJD iteration for every sequence of the batch (Sec. 4.1 Steps 1-4):
 *   inputs  [c[n-1], d_0 .. d_{W_eff-2}] at positions n-1 .. n+W_eff-2,
 *           W_eff = min(W, P + N - n);
 *   forward one pass; logits row k (stored in cfg.dtype) predicts position n+k;
 *   verify  acc_k = u_k < min(1, p_k[d_k] / q_k[d_k]) scanned left to right (Eq. 1);
 *           at the first rejected row a: t ~ max(0, p_a - q_a) / sum (Eq. 2),
 *           fixed at once after d_0..d_{a-1}; rows k > a: d'_k ~ p_k (Eq. 3);
 *   slide   the re-drawn tokens move left by the number of fixed tokens, new
 *           slots are initialised (Sec. 4.2), rejected keys/values are
 *           rolled back (overwritten by the next step).
 * Sampling is by inverse CDF in token order.  Asynchronous on the stream.
 * A finished sequence reports n_committed = 0 and SJD_FLAG_DONE.
 * Errors: STATE (no prefill), BAD_ARG, CUDA.
 */
int sjd_step(sjd_ctx *ctx, const sjd_step_out *out, void *cuda_stream);

/* Current window (drafts, their laws, n) without stepping; fields n_accepted,
 * n_committed, committed and flags of `out` are not written. */
int sjd_get_window(sjd_ctx *ctx, const sjd_step_out *out, void *cuda_stream);

/* The output of Algorithm 1: the tokens fixed so far.  tokens: device int32 [images][row_stride], image i
 * receives its prompt followed by the tokens it has accepted (under guidance: the conditional stream, which
 * holds the same accepted tokens as the unconditional one); entries past its count are not written.
 * counts: device int32 [images], prompt length + accepted tokens of each image (may be null).
 * images = the batch of the pre-fill (half of it under guidance).  Asynchronous on the stream.
 * Errors: STATE (no prefill), BAD_ARG, CAPACITY (row_stride below a sequence's prompt + n_generate). */
int sjd_get_tokens(sjd_ctx *ctx, int32_t *tokens, int row_stride, int32_t *counts, void *cuda_stream);

/* Copy the stored logits of the last step, [batch][window][vocab] in cfg.dtype,
 * to dst (device or host); for parity checks.  Errors: STATE, CAPACITY (bytes too small). */
int sjd_peek_logits(sjd_ctx *ctx, void *dst, size_t bytes, void *cuda_stream);

/*
 * The verification of Step 3 in isolation (Eqs. 1-3) on caller-supplied
 * logits.  logits_cur / logits_prev: device [batch][window][vocab] of
 * logits_dtype (this iteration's rows; the rows the drafts were drawn from);
 * draft: device int32 [batch][window]; q_kind: device int32 [batch][window]
 * or NULL (all SJD_Q_ROW); base_pos: device int32 [batch], absolute position
 * of window slot 0 (Philox counter), or NULL (all 0).  Outputs as sjd_step:
 * `draft` receives the re-drawn tokens of rows a+1.. left-aligned (no new
 * slots are initialised), total_committed = base_pos + n_committed.
 * ws: device scratch of sjd_verify_workspace_bytes(batch, window) bytes.
 * Errors: BAD_ARG, CAPACITY (ws too small, window > 64, vocab too large), CUDA.
 */
size_t sjd_verify_workspace_bytes(int batch, int window);
int sjd_verify(int batch, int window, int vocab, int logits_dtype, const void *logits_cur,
               const void *logits_prev, const int32_t *draft, const int32_t *q_kind,
               const int32_t *base_pos, const sjd_sample_cfg *sample, uint32_t step,
               const sjd_step_out *out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sjd_verify without a scratch argument, for callers that cannot allocate device memory: code that
 * runs where cudaMalloc is forbidden or would stall the device (inside a serving loop with a latency
 * budget, in a host thread that owns no allocator, in a plug-in that is handed only its input and
 * output buffers).  (The paper has no counterpart; this is a packaging variant of the same kernel.)
 *
 * Same arguments, outputs and results as sjd_verify, minus ws / ws_bytes.  The per-row scratch lives
 * in a fixed array inside the library image, SJD_VERIFY_STATIC_MAX_ROWS rows (about 130 KB); every
 * GPU that loads the library holds that array until the process exits.  The call performs no
 * cudaMalloc / cudaFree and calls no allocating routine; inputs and outputs stay the caller's.
 *   - Limits: batch * window <= SJD_VERIFY_STATIC_MAX_ROWS and batch <= SJD_VERIFY_STATIC_MAX_BATCH,
 *     else SJD_ERR_CAPACITY (nothing is launched).
 *   - Every call looks up the array's device address for the current device (a host-side query of
 *     the loaded library, no allocation).  The first call on a device also makes the CUDA runtime load
 *     the library's device code there: make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps the previous call's contents; the call
 *     clears the counters that must start at zero.  Two calls that overlap on the GPU (different
 *     streams, or different threads of the same process on one device) race on it:
 *     serialise them.  sjd_verify with separate workspaces has no such restriction.
 */
#define SJD_VERIFY_STATIC_MAX_ROWS 2048
#define SJD_VERIFY_STATIC_MAX_BATCH 256
int sjd_verify_static(int batch, int window, int vocab, int logits_dtype, const void *logits_cur,
                      const void *logits_prev, const int32_t *draft, const int32_t *q_kind,
                      const int32_t *base_pos, const sjd_sample_cfg *sample, uint32_t step,
                      const sjd_step_out *out, void *cuda_stream);

/*
 * One projection of the forward pass (Sec. 4.1 Step 2) in isolation, on the tensor-core
 * weight-streaming kernel sjd_step uses for bf16 models:
 *     out[m][n] (+)= sum_k x[m][k] * w[n][k]      (fp32 accumulation)
 * x: device fp32 [M][K] (split internally into bf16 hi + lo parts, so activations keep ~16 bits of
 * mantissa); w: device bf16 [N][K]; out: device fp32 [M][N], overwritten (accumulate = 0) or added
 * to (accumulate != 0).  Covered shapes: 1 <= M <= 1024 (above 128 rows the launch is cut into token
 * slabs of at most 128 rows that share each weight tile through L2), N a multiple of 128, K a
 * multiple of 64, compute capability 10.x; anything else returns SJD_ERR_UNSUPPORTED (sjd_step then uses its generic
 * kernel).  ws: device scratch of sjd_gemm_workspace_bytes(M, N, K), 256-byte aligned; after the stream
 * has drained its first int32 is 0, or non-zero if a bounded device-side wait ran out.
 * Errors: BAD_ARG, UNSUPPORTED, CAPACITY (ws too small), CUDA.
 */
size_t sjd_gemm_workspace_bytes(int M, int N, int K);
int sjd_gemm(int M, int N, int K, const float *x, const void *w, float *out, int accumulate, void *ws,
             size_t ws_bytes, void *cuda_stream);

/*
 * The window-causal attention of the forward pass (Sec. 3.2 / Sec. 4.1 Step 2) in isolation, on the
 * tensor-core split-KV kernel sjd_step uses for bf16 caches: query row m = b * window + k, at absolute
 * position in_pos[m] (-1: inactive row, output zeros), attends cache rows 0 .. in_pos[m] of sequence b:
 *     out[m][h] = softmax(q[m][h] . K[b][h / (H/KVh)][0..pos]^T / sqrt(head_dim)) V[b][...][0..pos]
 * q, out: device fp32 [batch*window][n_heads*head_dim]; kv_cache: device bf16
 * [batch][K|V][n_kv_heads][max_seq][head_dim], finite everywhere (rows beyond the positions are read
 * and masked); in_pos: device int32 [batch*window].  Covered: head_dim 64 or 128, window <= 64,
 * compute capability >= 9; anything else returns SJD_ERR_UNSUPPORTED.  ws: device scratch of
 * sjd_attention_workspace_bytes(...), 256-byte aligned; its first int32 is non-zero after the stream
 * has drained if a bounded device-side wait ran out.
 * Errors: BAD_ARG, UNSUPPORTED, CAPACITY, CUDA.
 */
size_t sjd_attention_workspace_bytes(int batch, int window, int n_heads, int head_dim);
int sjd_attention(int batch, int window, int n_heads, int n_kv_heads, int head_dim, int max_seq, const float *q,
                  const void *kv_cache, const int32_t *in_pos, float *out, void *ws, size_t ws_bytes,
                  void *cuda_stream);

/*
 * Which kernels the steps of a pre-filled context run (the forward pass of Sec. 4.1 Step 2 has two
 * implementations: the tensor-core pipeline for bf16 models whose projection widths are multiples
 * of 128 with inner sizes that are multiples of 64, and generic FMA kernels, roughly 50 times slower
 * on the projections, for everything else).  Host-side query, nothing is launched.
 * Errors: BAD_ARG, STATE (no prefill yet: the answer depends on batch and window).
 */
typedef struct {
  int32_t tensor_core_projections; /* 1: tcgen05 weight-streaming GEMM + fused consumers; 0: generic kernels */
  int32_t tensor_core_attention;   /* 1: TMA-staged split-KV tensor-core attention; 0: generic kernel       */
  int32_t step_graph;              /* 1: a step is replayed as one captured CUDA graph                       */
  int32_t rows_per_step;           /* batch * window rows per forward pass                                    */
} sjd_info;
int sjd_get_info(sjd_ctx *ctx, sjd_info *info);

/* Synchronises the context's last stream and returns SJD_OK, SJD_ERR_DEVICE_TIMEOUT
 * or SJD_ERR_CUDA according to the device status word. */
int sjd_last_device_status(sjd_ctx *ctx);

/* cudaError_t of the last failed CUDA call made on behalf of this thread (0 if none). */
int sjd_last_cuda_error(void);

/* Number of kernels this library has launched in this process (all contexts, all calls). */
int64_t sjd_launch_count(void);

/*
 * Diagnostics: where the time of Step 2 / Step 3 goes.  sjd_trace(ctx, 1) zeroes the totals and
 * makes every following sjd_step bracket each kernel launch with CUDA events on the caller's
 * stream and end with a stream synchronisation (so traced steps are slower and must not be the
 * ones a throughput figure is taken from); sjd_trace(ctx, 0) switches it off.  sjd_trace_read
 * returns, per class {0: projection GEMMs, 1: attention, 2: verify + window slide, 3: the rest},
 * the summed device milliseconds and launch counts (host arrays of 4), and the weight bytes the
 * traced GEMM launches had to stream (out_features * in_features * element size, summed).
 */
int sjd_trace(sjd_ctx *ctx, int enable);
int sjd_trace_read(sjd_ctx *ctx, double *ms, int64_t *launches, double *gemm_weight_bytes);

void sjd_destroy(sjd_ctx *ctx);
const char *sjd_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SJD_H_ */
