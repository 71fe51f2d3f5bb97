/*
 * eesd.h -- C ABI of the EESD decode-round library for NVIDIA B200 (sm_100a).
 *
 * EESD = Early-exiting Speculative Decoding (Liu et al., arXiv 2406.03853).  One decode
 * round drafts K tokens with the draft model of Eq. 1 (first N decoder layers of the target
 * model, one early-exit decoder layer, RMSNorm, own vocabulary head), then verifies them in
 * ONE forward pass of the target model over K+1 rows (Algorithm 1, verification step) and
 * applies lossless speculative acceptance; a Thompson-sampling controller with a Beta
 * posterior (Sec. 3.3, Eq. 3-4, Algorithm 2) decides when drafting stops.
 *
 * Conventions
 *   - every function returns an int status: EESD_OK (0) or a negative EESD_ERR_* value; no
 *     function throws, aborts or traps the device.  eesd_strerror() gives a text.
 *   - "device" pointers are CUDA global-memory addresses of the current device; "host"
 *     pointers are ordinary process memory.  The library never allocates or frees device
 *     memory: all of it is passed in through eesd_buffers and stays owned by the caller, who
 *     must keep it alive until eesd_destroy().
 *   - matrices are row-major [out_features][in_features] (the input dimension is contiguous).
 *   - batch size is 1 sequence per context (the paper's setting, Sec. 4.1); the standalone
 *     acceptance entry points take a batch of independent sequences.
 *   - all work is enqueued on the CUDA stream given at eesd_init(); calls that return
 *     host-visible results synchronise that stream before returning.
 *   - a context is not thread-safe; use one per host thread / stream.  Contexts on different
 *     host threads may be created and used concurrently (one-time set-up inside the library is
 *     guarded).
 */
#ifndef EESD_H
#define EESD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    EESD_OK = 0,
    EESD_ERR_BADARG = -1,      /* null pointer, non-positive size, inconsistent shape         */
    EESD_ERR_NOMEM = -2,       /* a caller-provided buffer is smaller than required            */
    EESD_ERR_CUDA = -3,        /* a CUDA runtime call failed (see eesd_last_cuda_error)        */
    EESD_ERR_STATE = -4,       /* call not valid in the current state (e.g. verify w/o draft)  */
    EESD_ERR_CTX_FULL = -5,    /* the round would exceed max_ctx or the KV page pool           */
    EESD_ERR_RNG = -6,         /* a uniform stream is missing or exhausted                     */
    EESD_ERR_DEVICE = -7,      /* a kernel reported an error word (bad token id, bounded wait) */
    EESD_ERR_UNSUPPORTED = -8  /* shape outside what the kernels support                       */
};

enum { EESD_F32 = 0, EESD_BF16 = 1 };
enum { EESD_CTRL_FIXED_K = 0, EESD_CTRL_BETA_TS = 1, EESD_CTRL_CALI_TS = 2 };
enum { EESD_TS_RULE_PAPER = 0, EESD_TS_RULE_SINGLE_FAILURE = 1 };

#define EESD_MAX_ROWS 16 /* most token rows one pass processes (k_cap + 1 <= 16) */

/* Model and round configuration (plain data, copied by eesd_init). */
typedef struct eesd_config {
    int32_t d_model;      /* d: residual width (multiple of 8)                                  */
    int32_t n_heads;      /* H: query heads                                                     */
    int32_t n_kv_heads;   /* H_kv: key/value heads (H % H_kv == 0)                              */
    int32_t head_dim;     /* D: 64 or 128                                                       */
    int32_t ffn_dim;      /* F: SwiGLU hidden width (multiple of 8)                             */
    int32_t vocab;        /* V                                                                  */
    int32_t n_layers;     /* L: decoder layers of the target model                              */
    int32_t n_early;      /* N: first layers shared by the draft model (Sec. 3.1), 1 <= N <= L  */
    int32_t dtype;        /* EESD_F32 or EESD_BF16: weights and KV cache (activations are fp32) */
    int32_t tie_exit_head;/* 1: the exit head W of Eq. 1 is the target LM head (same storage)   */
    float rms_eps;        /* RMSNorm epsilon                                                    */
    float rope_theta;     /* rotary base; pairs (2i, 2i+1) turn by pos * theta^(-2i/D)          */
    int32_t page_tokens;  /* tokens per KV page (power of two, 8..128)                          */
    int32_t max_ctx;      /* most tokens a sequence may hold (prompt + generated + drafts);
                             at most 12288, and 8192 for an fp32 cache with 128-token pages         */
    int32_t k_cap;        /* most draft tokens per round, 1 <= k_cap <= EESD_MAX_ROWS - 1       */
    float temperature;    /* 0: greedy (draft top-1, accept while equal to target top-1)        */
    int32_t controller;   /* EESD_CTRL_FIXED_K, EESD_CTRL_BETA_TS or EESD_CTRL_CALI_TS                */
    int32_t fixed_k;      /* draft length for EESD_CTRL_FIXED_K                                 */
    int32_t alpha0;       /* Beta prior (Algorithm 2, initialisation); positive integers        */
    int32_t beta0;
    int32_t ts_update_rule; /* EESD_TS_RULE_PAPER: r = |Q_v|-1, n = min(|Q_v|+1, |Q_d|)          */
    /* EESD_CTRL_CALI_TS only (Sec. 3.3 "TS with Calibration", Algorithm 3): the assumed error of
     * the model's prediction, the assumed deviation of a round's sample mean, and the initial
     * observed mean theta_hat_0; sigmas must be positive */
    float cali_sigma_m, cali_sigma_s, cali_theta0;
    /* Tree verification (appendix "Implement Tree Attention": several draft candidates per
     * position, only the one equal to the target's top-1 token is kept).  0 or 1: off.  2..4:
     * beside the draft's greedy chain x_1..x_K, the tree_width - 1 next-best tokens of each draft
     * step (by logit, lower id first among equals) enter the verification pass as leaves of that
     * depth; a leaf sees the cache, the chain before its depth and itself.  The target's top-1
     * after the accepted path is compared with the candidates of the next depth: the chain token
     * continues, a leaf is kept and ends the round (next token = the target's top-1 after that
     * leaf), neither ends the round with the target's token.  The paper fixes no tree shape: this
     * one is a choice.  Needs temperature 0, a controller other than EESD_CTRL_CALI_TS and
     * 1 + k_cap * tree_width <= EESD_MAX_ROWS (else UNSUPPORTED / BADARG); a round of K drafts
     * uses 1 + K * tree_width cache rows past the context before it is cut back, so
     * eesd_generate / eesd_decode want n_prompt + max_new + tree_width <= max_ctx (CTX_FULL
     * otherwise) and shorten the last rounds' drafts to what fits. */
    int32_t tree_width;
    /* Early-exit layers of the draft model (the paper's experiment on the number of exit layers; its
     * method and Eq. 1 use one).  0 or 1: one.  2..4: a stack of that many decoder layers on H^N, stored
     * one after the other from eesd_layout.exit_layer on, each with its own cache slot; prefill and
     * verification then also run all exit layers but the last on their rows (exit layer e needs the
     * output of exit layer e - 1 to form its keys / values), so each costs that many more layers. */
    int32_t n_exit_layers;
} eesd_config;

/* Byte offsets inside the weight buffer.  A decoder layer holds, in this order:
 *   g_attn f32[d] | wqkv [(H+2H_kv)D][d] (q heads, k heads, v heads) | wo [d][H*D] |
 *   g_ffn f32[d]  | wgu [2F][d] (gate rows then up rows) | wd [d][F]
 * matrices in the configured dtype, gains always fp32.  Storage of a matrix W [R][K] ([out][in]):
 * row-major when tiled == 0 (fp32 models, shapes the tensor-core tiles do not divide); when
 * tiled == 1 (bf16 models whose projection shapes are multiples of 128 rows and 64 columns),
 * as [R/128][K/64] tiles of [128][64] elements, each tile 16 KB contiguous:
 *   element (r, k) sits at ((r/128 * (K/64) + k/64) * 128 + r%128) * 64 + k%64.
 * The weight stream then reads whole contiguous tiles (measured 1 to 4 % faster than 128-byte
 * pieces of 128 rows).  The embedding [V][d] is always row-major (it is gathered by rows).  Target layer l starts at
 * layer0 + l * layer_stride; the early-exit layer (Eq. 1, Transformer^e) at exit_layer. */
typedef struct eesd_layout {
    size_t embed;        /* [V][d] token embedding                                              */
    size_t layer0, layer_stride;
    size_t off_g_attn, off_wqkv, off_wo, off_g_ffn, off_wgu, off_wd; /* within a layer          */
    size_t final_norm;   /* f32[d]                                                              */
    size_t lm_head;      /* [V][d]                                                              */
    size_t exit_layer;   /* the early-exit layer(s): n_exit_layers decoder layers, layer_stride apart */
    size_t exit_norm;    /* f32[d], the RMSNorm before the exit head                            */
    size_t exit_head;    /* [V][d]; equals lm_head when tie_exit_head                           */
    size_t cali_w;       /* EESD_CTRL_CALI_TS only (else 0): W^1..W^10 of Eq. 5, [10][d][d]           */
    size_t cali_wp;      /* EESD_CTRL_CALI_TS only (else 0): W_p of Eq. 5, f32 [2][2d]                */
    size_t total_bytes;
    size_t tiled;        /* 1: every [R][K] matrix except the embedding is stored TILE-MAJOR (below)  */
} eesd_layout;

typedef struct eesd_sizes {
    size_t weights_bytes;
    size_t kv_page_bytes;   /* bytes of ONE page across all L + n_exit_layers cache slots       */
    int64_t min_pages;      /* pages needed to hold max_ctx tokens                              */
    size_t workspace_bytes;
} eesd_sizes;

/* Caller-owned device memory.  kv_pool holds P = floor(kv_bytes / kv_page_bytes) pages laid
 * out [slot 0..L+E-1][page 0..P-1][K|V][H_kv] blocks of page_tokens * D elements; slots L.. are the
 * caches of the E early-exit layers.  The element order inside a block is an internal format (the library
 * writes and reads the pool itself): for a bf16 cache both blocks are grids of 8 x 8 element
 * groups, [token/8][D/8][8][8], keys with a group's 8 tokens as rows, values with its 8 dimensions
 * as rows, which is the form the tensor cores take an operand in; for an fp32 cache keys are
 * [D/2][page_tokens][2] and values [page_tokens][D] with 16-byte chunks permuted by the token.
 * The workspace must be zero-filled by the caller before eesd_init; eesd_init zero-fills the KV
 * pool itself (the attention kernel relies on the pool never holding a non-finite value). */
typedef struct eesd_buffers {
    void *weights;   size_t weights_bytes;
    void *kv_pool;   size_t kv_bytes;
    void *workspace; size_t workspace_bytes;
} eesd_buffers;

/* Host arrays of uniforms in [0,1) of the form m * 2^-24 (random numbers are inputs, never
 * drawn inside the library).  u_draft[p] / u_accept[p]: used when the token that would take
 * context position p is drafted / tested; u_resample[p]: used by the round whose first
 * drafted token takes position p; each needs max_ctx entries.  u_ctrl is consumed in order by
 * the controller (alpha + beta + 1 values per decision). */
typedef struct eesd_uniforms {
    const float *u_draft, *u_accept, *u_resample;
    const float *u_ctrl; int64_t n_ctrl;
} eesd_uniforms;

typedef struct eesd_round { int32_t k, n_accept, next_token; } eesd_round;

/* Counters of one eesd_generate / eesd_decode call.  v_d = accepted / drafted and r_d = accepted /
 * emitted are the paper's acceptance rate and draft proportion (metrics paragraph of Sec. 4.1).
 * Times follow the buckets of the paper's time-breakdown table (drafting, verification, sampling,
 * others), with the prompt pass kept apart:
 *   ms_prefill   device time of the prompt pass (CUDA events; 0 for eesd_decode)
 *   ms_draft     device time of the draft steps (draft model + token choice)
 *   ms_verify    device time of the verification passes, without their acceptance step
 *   ms_sampling  the acceptance step (device: fused softmax / accept / resample kernel, or the tree
 *                walk), the calibrated controller's predictor steps (device), and the controller's
 *                draws on the host (host clock)
 *   ms_other     what is left of ms_total: synchronisation gaps, copies, host bookkeeping
 *   ms_total     wall time of the call on the host clock; the five above add up to it */
typedef struct eesd_stats {
    int64_t rounds, drafted, accepted, emitted;
    double ms_prefill, ms_draft, ms_verify, ms_total;
    int64_t kernel_launches;
    int64_t alpha, beta;                               /* posterior after the last round         */
    int64_t leaves_kept;                               /* tree verification: rounds that kept a leaf */
    double ms_sampling, ms_other;
} eesd_stats;

typedef struct eesd_ctx eesd_ctx;

const char *eesd_strerror(int status);
/* Text of the last CUDA error seen by this context (empty string if none). */
const char *eesd_last_cuda_error(const eesd_ctx *ctx);

/* Fills the weight-buffer layout for a configuration.  EESD_ERR_BADARG on invalid shapes. */
int eesd_weight_layout(const eesd_config *cfg, eesd_layout *out);
/* Sizes of the three device buffers eesd_init needs for a configuration. */
int eesd_required_bytes(const eesd_config *cfg, eesd_sizes *out);

/* Creates a context over caller-owned device buffers (weights already filled by the caller).
 * `cuda_stream` is a cudaStream_t (borrowed; NULL = default stream).  Builds the rotary table
 * and the KV page allocator; enqueues small set-up kernels on the stream.
 * Errors: BADARG (shape), NOMEM (a buffer too small), UNSUPPORTED, CUDA. */
int eesd_init(const eesd_config *cfg, const eesd_buffers *bufs, void *cuda_stream, eesd_ctx **out);
/* Frees host state only. */
int eesd_destroy(eesd_ctx *ctx);
/* Forgets the sequence: context length 0, all KV pages free, posterior back to the prior. */
int eesd_reset(eesd_ctx *ctx);

/* Algorithm 1, initialisation of Q_g with the prompt: runs prompt tokens 0..n-2 through all L
 * target layers (and writes the early-exit layer's keys/values for them), leaving the last
 * prompt token pending, i.e. it is the first row of the next draft step and verify pass.
 * `prompt` is a host pointer, borrowed for the call.  Resets the sequence first.
 * Errors: BADARG (n_prompt < 1 or a token id outside [0, V)), CTX_FULL. */
int eesd_prefill(eesd_ctx *ctx, const int32_t *prompt, int n_prompt);

/* Algorithm 1, draft loop body (Eq. 1): k more draft steps of the current round.  Each step
 * feeds the newest token through the first N layers (writing their shared KV rows) and the
 * early-exit layer, and picks x_i = argmax q_i (temperature 0) or x_i ~ softmax(q_i / T) with
 * uniform u_draft[i] (host array of k values, may be NULL when greedy).  The draft logits stay
 * on the device for verification.  out_tokens (host, k entries, may be NULL) receives the
 * tokens.  May be called repeatedly within a round, so a host controller can interleave.
 * Errors: STATE (no prefill), CTX_FULL (round longer than k_cap or context full), RNG. */
int eesd_draft(eesd_ctx *ctx, int k, const float *u_draft, int32_t *out_tokens);

/* Algorithm 1, verification step with lossless acceptance: one pass of the K+1 rows
 * (pending token, x_1..x_K) through all L layers against the KV cache, then for i = 1..K
 * accept x_i iff u_accept[i-1] * q_i(x_i) < p_i(x_i); at the first rejection j the next token is
 * drawn from normalize(max(0, p_j - q_j)), with no rejection from p_{K+1}, both with
 * u_resample.  Greedy: accept while x_i = argmax p_i, next token = argmax of the first
 * disagreeing row.  KV rows of rejected tokens are rolled back (pages past the end freed).
 * Afterwards the context holds the accepted tokens plus next_token, which is pending.
 * u_accept: host array of K values (may be NULL when greedy).  Errors: STATE (nothing drafted).
 * With tree verification (eesd_config.tree_width > 1) the pass also holds the draft steps'
 * next-best tokens as leaves; n_accept then counts a kept leaf as an accepted draft, and the
 * token accepted at that depth is the leaf, not the one eesd_draft returned:
 * eesd_context_tokens shows what the context gained.  Errors: CTX_FULL when the tree rows do
 * not fit below max_ctx. */
int eesd_verify_accept(eesd_ctx *ctx, const float *u_accept, float u_resample,
                       int *n_accept, int32_t *next_token);

/* Algorithm 1 end to end: prefill, then rounds of {draft until the controller stops or k_cap,
 * verify, accept, posterior update (Eq. 3-4)} until max_new tokens exist; the output is cut to
 * exactly max_new tokens.  k_schedule (host, may be NULL) forces the draft length of round r
 * to k_schedule[r] for r < n_schedule (then the configured controller takes over).
 * `u` may be NULL only for greedy decoding with a fixed K.  out: host, max_new entries.
 * stats / trace / n_rounds may be NULL; trace receives at most trace_cap rounds.
 * One host<->device synchronisation per round (to read n_accept and the next token). */
int eesd_generate(eesd_ctx *ctx, const int32_t *prompt, int n_prompt, int max_new,
                  const int32_t *k_schedule, int n_schedule, const eesd_uniforms *u,
                  int32_t *out, eesd_stats *stats, eesd_round *trace, int trace_cap, int *n_rounds);

/* ---- additions beyond the five calls above (testing and measurement) ---- */

/* The decode loop of eesd_generate without its prefill: continues from the current context
 * (after eesd_prefill, or a previous eesd_decode / eesd_verify_accept) for max_new more tokens.
 * Same arguments and errors as eesd_generate; STATE if no prefill or a round is half drafted. */
int eesd_decode(eesd_ctx *ctx, int max_new, const int32_t *k_schedule, int n_schedule,
                const eesd_uniforms *u, int32_t *out, eesd_stats *stats, eesd_round *trace,
                int trace_cap, int *n_rounds);

/* Context length in tokens (including the pending one), and KV pages in use. */
int eesd_context_len(const eesd_ctx *ctx, int *n_tokens, int *pages_in_use);
/* Tokens first .. first + n - 1 of the context (prompt, accepted tokens, pending token) into
 * out (host).  With tree verification this is how the step API shows which candidate a round
 * kept.  BADARG if the range passes the end of the context. */
int eesd_context_tokens(const eesd_ctx *ctx, int first, int n, int32_t *out);
/* Posterior parameters of the controller. */
int eesd_posterior(const eesd_ctx *ctx, int64_t *alpha, int64_t *beta);

/* Thompson sampling with calibration (Sec. 3.3, Eq. 5-8, Algorithm 3; EESD_CTRL_CALI_TS).
 * eesd_generate / eesd_decode then run the draft loop step by step: after every draft step
 * the device evaluates the predictor of Eq. 5,
 *     theta_M = softmax(W_p [W^i H^(T) ; H^(D)])[1],   i = min(draft step, 10),
 * with H^(T) the target's residual stream after its last layer at the last position it has
 * processed (the row whose logits produced the pending token; zeros before any pass) and H^(D)
 * the draft model's residual stream after the early-exit layer of that step; the host reads the
 * one float back (a stream synchronisation per draft step, which this controller cannot avoid),
 * forms the posterior of Eq. 6-7 from theta_M, the observed mean theta_hat and the number of
 * verifications n, draws theta ~ N(mu, sigma^2) (Box-Muller on two controller uniforms) and
 * chi ~ Bernoulli(theta) (a third).  After a verification theta_hat <- (theta_hat (N + 1) + r) /
 * (N + n_r + 1) with r successes in n_r verified drafts (those of Eq. 3-4) and N the verified
 * drafts before: the observed sample mean, theta_hat_0 counting as one observation.
 *
 * eesd_cali_predict: theta_M for the latest draft step of the round being drafted (for callers
 * driving eesd_draft / eesd_verify_accept themselves); host pointer; synchronises the stream.
 * STATE unless the controller is EESD_CTRL_CALI_TS and at least one step has been drafted.
 * eesd_cali_state: theta_hat, verifications so far, verified drafts so far.
 * eesd_cali_posterior: Eq. 6-7 on the host (no context needed); BADARG for non-positive sigmas. */
int eesd_cali_predict(eesd_ctx *ctx, float *theta_m);
int eesd_cali_state(const eesd_ctx *ctx, double *theta_hat, int64_t *n_verify, int64_t *n_trials);
int eesd_cali_posterior(double theta_m, double theta_hat, int64_t n, double sigma_m, double sigma_s,
                        double *mu, double *variance);

/* The host-side controller arithmetic, exported so that it can be checked on its own (no context,
 * no device).  These are the functions eesd_generate / eesd_decode / eesd_verify_accept call.
 * eesd_ts_decide (Algorithm 2, draft loop): theta ~ Beta(alpha, beta), chi ~ Bernoulli(theta), from
 * alpha + beta + 1 uniforms u[*cursor ...] (host): theta = X / (X + Y), X = sum of -ln u over the
 * first alpha of them, Y over the next beta, chi = [next uniform < theta]; a zero uniform counts
 * as 2^-25.  Returns chi (0 or 1) and advances *cursor; RNG when fewer than alpha + beta + 1
 * uniforms are left (cursor unchanged), BADARG for non-positive parameters.  theta_out may be NULL.
 * eesd_ts_posterior_update (Eq. 3-4; Algorithm 2, update steps) after a round that drafted
 * n_draft = |Q_d| tokens and added q_v = |Q_v| tokens (accepted drafts + the target's own):
 * r = q_v - 1, n = min(q_v + 1, n_draft) (EESD_TS_RULE_PAPER) or min(q_v, n_draft)
 * (EESD_TS_RULE_SINGLE_FAILURE); alpha += r, beta += n - r.  BADARG unless 1 <= q_v <= n_draft + 1.
 * eesd_cali_decide (Algorithm 3, draft loop): theta = mu + sqrt(variance) * sqrt(-2 ln u_0) *
 * cos(2 pi u_1), chi = [u_2 < theta], three uniforms from u[*cursor ...]. */
int eesd_ts_decide(int64_t alpha, int64_t beta, const float *u, int64_t n_u, int64_t *cursor, double *theta_out);
int eesd_ts_posterior_update(int64_t *alpha, int64_t *beta, int q_v, int n_draft, int rule);
int eesd_cali_decide(double mu, double variance, const float *u, int64_t n_u, int64_t *cursor, double *theta_out);

/* Declares that the KV cache already holds n_ctx - 1 valid rows (whatever bytes the pool
 * contains) and that `pending` is the pending token: allocates pages, sets the length.  Used to
 * time a verify pass against a cache of a chosen length without running a prefill. */
int eesd_assume_context(eesd_ctx *ctx, int n_ctx, int32_t pending);

/* One verification pass of M rows (tokens: host, M entries; row 0 replaces the pending token)
 * at the current position WITHOUT acceptance: logits stay in the context (eesd_logits), the
 * context length is unchanged afterwards.  The verify pass of Algorithm 1 at a forced M.
 * Asynchronous: enqueues on the context's stream and returns. */
int eesd_verify_only(eesd_ctx *ctx, const int32_t *tokens, int M);

/* Device pointers of the fp32 logits of the last verify pass ([rows][V], which = 0) and of
 * the current round's draft steps ([k][V], which = 1). */
int eesd_logits(const eesd_ctx *ctx, int which, const float **device_ptr);

/* When set (device buffer of (L + 2) * EESD_MAX_ROWS * d floats, or NULL to stop), every
 * pass stores the residual stream after the embedding (index 0), after target layer l
 * (index l + 1) and, in draft steps, after the early-exit layer (index L + 1) as
 * [index][row][d] fp32. */
int eesd_capture_hidden(eesd_ctx *ctx, float *device_buf, size_t bytes);

/* Bound of the waits inside the kernels.  Every wait of a kernel on data in flight (a bulk copy
 * into shared memory, a tensor-core operation) polls at most `polls` times (a second or two's worth
 * by default; 0xffffffff restores the default); a wait that runs out makes its thread block raise
 * the context's error word, skip the rest of its work, let the copies it has already requested land
 * and return, and the call that reads results next returns EESD_ERR_DEVICE.  polls = 0 makes the
 * first wait of every block give up at once: no result is produced, nothing is left in flight, and
 * the error path can be exercised without stalling anything.
 * eesd_clear_device_error: zeroes the error word and the counters a failed pass may have left half
 * counted, and forgets the sequence (as eesd_reset; in batch mode all sequences: the context is back in
 * single-sequence mode); the context is usable again afterwards. */
int eesd_set_wait_limit(eesd_ctx *ctx, uint32_t polls);
int eesd_clear_device_error(eesd_ctx *ctx);

/* ---- batch mode: several sequences decoded together -------------------------------------------
 * An extension: the paper decodes one sequence at a time (its experiments run at batch 1).  The
 * rows of a pass (at most EESD_MAX_ROWS) are shared by up to EESD_MAX_BATCH sequences, each with
 * its own KV pages (one pool), positions and tokens; every weight crosses HBM once per pass for
 * all of them.  A round drafts the same number K of tokens for every sequence that still owes
 * tokens (n * (K + 1) <= EESD_MAX_ROWS rows in its verification pass): K comes from the schedule
 * or from eesd_config.fixed_k; the controllers' per-sequence stopping rule (Algorithms 2-3) has
 * no batch counterpart and is not consulted.  Per sequence the result is what single-sequence
 * decoding with the same draft lengths and the same uniforms gives (Algorithm 1: drafting,
 * verification and acceptance of a sequence never look at another sequence).
 * Not with tree verification (UNSUPPORTED).  While batch mode is on,
 * the single-sequence calls that start or feed a sequence return STATE. */
#define EESD_MAX_BATCH 8
/* Enters batch mode with n_seq empty sequences (1..EESD_MAX_BATCH), or leaves it (n_seq = 0); either
 * way every sequence is forgotten and all KV pages are free afterwards. */
int eesd_batch_begin(eesd_ctx *ctx, int n_seq);
/* eesd_prefill for sequence `seq` of the batch (same arguments and errors). */
int eesd_batch_prefill(eesd_ctx *ctx, int seq, const int32_t *prompt, int n_prompt);
/* Rounds of {K draft steps on one row per sequence, one verification pass of K + 1 rows per sequence,
 * acceptance of all sequences in one kernel launch} until every sequence has max_new new tokens; a
 * sequence that has them leaves the rounds.  k_schedule[r] (host, may be NULL) is the draft length of
 * round r < n_schedule, then fixed_k; either is cut to what the pass rows, k_cap and the contexts allow.
 * u: one eesd_uniforms per sequence (host; may be NULL when greedy; u_ctrl unused).
 * out: host, [n_seq][max_new].  stats: sums over the sequences (rounds = rounds of the batch).
 * trace (may be NULL): [n_seq][trace_cap]; n_rounds (may be NULL): [n_seq] rounds each sequence took part in.
 * Errors: BADARG, STATE (batch mode off or a sequence without prompt), RNG, CTX_FULL, DEVICE. */
int eesd_batch_decode(eesd_ctx *ctx, int max_new, const int32_t *k_schedule, int n_schedule,
                      const eesd_uniforms *u, int32_t *out, eesd_stats *stats, eesd_round *trace,
                      int trace_cap, int *n_rounds);
/* Context length (pending token included) and KV pages of one sequence of the batch. */
int eesd_batch_context_len(const eesd_ctx *ctx, int seq, int *n_tokens, int *pages_in_use);
/* Test and measurement hooks, the batch forms of eesd_verify_only / eesd_assume_context: one pass of the
 * target model over m rows per sequence (tokens: host, [n_seq][m], n_seq * m <= EESD_MAX_ROWS) at the end
 * of each sequence's context, logits of row b * m + i in eesd_logits(.., 0, ..); and a sequence declared
 * to hold n_ctx tokens whose cache rows are whatever the pool holds. */
int eesd_batch_verify_only(eesd_ctx *ctx, const int32_t *tokens, int m);
int eesd_batch_assume_context(eesd_ctx *ctx, int seq, int n_ctx, int32_t pending);

/* How the attention kernel of a pass would cut a context of ctx_len tokens (host arithmetic, no
 * device needed): pages per thread block and thread blocks ("slices") per KV head, for `pairs`
 * (query head, new row) pairs per KV head on a device of n_sm multiprocessors.  A slice count
 * above 64 cannot be merged; configurations that could need one are refused by eesd_init
 * (UNSUPPORTED), and this call returns UNSUPPORTED for such a ctx_len. */
int eesd_attention_plan(int dtype, int ctx_len, int page_tokens, int n_kv_heads, int pairs, int n_sm,
                        int *pages_per_block, int *n_slices);

/* Kernel launches issued by this context since creation. */
int eesd_launch_count(const eesd_ctx *ctx, int64_t *n);

/* Standalone fused softmax / accept / residual-resample over a batch of B independent
 * sequences (the acceptance step of eesd_verify_accept).  All pointers are device pointers:
 * p_logits [B][K+1][V] f32, q_logits [B][K][V] f32, tokens [B][K] i32 (the drafted x_i),
 * u_accept [B][K], u_resample [B]; outputs n_accept [B], next_token [B] (i32).  scratch: 16-byte
 * aligned (BADARG otherwise), at least eesd_accept_scratch_bytes(B, K) bytes, contents irrelevant
 * (the call clears what it needs).  A drafted token id outside [0, V) is rejected at its position
 * (it cannot have been drawn from q); no logit is read for it.  Asynchronous on `cuda_stream`.
 * Errors: BADARG, NOMEM (scratch), RNG. */
size_t eesd_accept_scratch_bytes(int B, int K);
int eesd_accept_resample(void *cuda_stream, const float *p_logits, const float *q_logits,
                         const int32_t *tokens, const float *u_accept, const float *u_resample,
                         int B, int K, int V, float temperature, void *scratch, size_t scratch_bytes,
                         int32_t *n_accept, int32_t *next_token);

/* The same acceptance step for callers that cannot hand over device scratch memory.  The paper
 * has no counterpart: this exists for deployment reasons only.  Some hosts of this library may
 * not allocate on the device at the point where they verify a round: code running inside a
 * frozen memory plan (a serving engine that sized every buffer at start-up and forbids
 * allocation on the request path), plug-ins that are given only their input and output
 * tensors, or processes whose allocator must not be re-entered from the calling thread.  For
 * them the scratch lives inside the library as a fixed device array of about 80 KB, present in
 * every GPU context that loads the library until the process exits.
 * Limits: B <= EESD_STATIC_ACCEPT_MAX_BATCH and B * (2K + 1) <= EESD_STATIC_ACCEPT_MAX_ROWS;
 * larger problems return EESD_ERR_NOMEM (use eesd_accept_resample with your own scratch).
 * Inputs, outputs, arithmetic and results are exactly those of eesd_accept_resample.  The call
 * performs no device allocation or free.  The first call on each device looks up the array's
 * device address (one cudaGetSymbolAddress, with that device current; the address is kept for
 * the life of that device's primary context, so do not reset the device while the library is in
 * use); make that first call before any stream capture.  All calls share the one array and it keeps the previous call's
 * contents (the call re-zeroes what has to start at zero): two calls whose kernels may overlap
 * on the GPU (different streams, no ordering between them) race on it and must be avoided. */
#define EESD_STATIC_ACCEPT_MAX_BATCH 1024
#define EESD_STATIC_ACCEPT_MAX_ROWS 4800
int eesd_accept_resample_static(void *cuda_stream, const float *p_logits, const float *q_logits,
                                const int32_t *tokens, const float *u_accept, const float *u_resample,
                                int B, int K, int V, float temperature,
                                int32_t *n_accept, int32_t *next_token);

/* The skinny projection used by every weight-streaming step of a pass (QKV, attention output,
 * SwiGLU gate/up and down, vocabulary heads): out[m][r] = sum_k A[m][k] * W[r][k] for
 * M <= EESD_MAX_ROWS rows.  A [M][K] fp32, W [R][K] in `dtype`, out [M][R] fp32, all device.
 * bf16 weights with R % 128 == 0 and K % 64 == 0 take the tensor-core path (the rows are split
 * into two bf16 terms first), everything else the SIMT path.  scratch: device, 256-byte
 * aligned, at least eesd_project_scratch_bytes(R, K) bytes; afterwards its first 4 bytes hold
 * an error word (0 = none).  Asynchronous on `cuda_stream`.  K must be a multiple of 8. */
size_t eesd_project_scratch_bytes(int R, int K);
int eesd_project_rows(void *cuda_stream, int dtype, const float *A, const void *W, float *out,
                      int M, int R, int K, void *scratch, size_t scratch_bytes);

/* Times the projection kernel of one kind (0 QKV, 1 attention output, 2 gate/up, 3 down) as
 * the passes launch it: once over every target layer's matrix untimed, then once more
 * bracketed by CUDA events on the context's stream.  Returns the mean device time per launch
 * and the weight bytes one launch streams.  Synchronises.  The activation content is whatever
 * the last pass left in the context. */
int eesd_time_projection(eesd_ctx *ctx, int which, int M, float *ms_per_launch, size_t *bytes_per_launch);

/* Draws one token per row: argmax (temperature 0) or x ~ softmax(logits / T) by inverse CDF
 * with u[b].  logits [B][V] f32, u [B] (may be NULL when greedy), out [B] i32; device pointers. */
int eesd_sample_rows(void *cuda_stream, const float *logits, const float *u, int B, int V,
                     float temperature, int32_t *out);

#ifdef __cplusplus
}
#endif
#endif /* EESD_H */
