/*
 * sfs.h — C ABI of libsfs: the per-step denoising hot path of SlowFast Sampling for masked-diffusion
 * language models, for NVIDIA B200 (sm_100a).
 *
 * One denoising step (paper Section 3.1, Eqs. 2-4) is
 *     logits = p_theta(prompt || partially masked response)        -> sfs_forward
 *     r_hat_i, c_i = argmax / max softmax probability per row       -> sfs_row_stats
 *     y^(k-1) = S(r_hat, y^(k), k)   with S the SlowFast rule        -> sfs_select
 * and sfs_generate runs the whole loop of Algorithm 1 on the device.
 *
 * Conventions
 *   * Every function returns an int32 status: SFS_OK (0) or a negative SFS_ERR_* code.  Nothing throws,
 *     aborts or traps the device.  sfs_last_error() gives a human-readable message for the last failure
 *     on the calling thread.
 *   * Pointers whose name starts with d_ are DEVICE pointers owned by the caller; all others are HOST
 *     pointers.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *     validate their arguments on the host, enqueue work on `stream` and return without synchronising,
 *     unless stated otherwise.
 *   * Tokens are int32 [B, S] row-major with S = P + L (prompt then response); `mask` is uint8 [B, S],
 *     1 = position still masked.  A "row" is a flat token index b*S + pos.  Response positions are
 *     0-based: i = pos - P.
 *   * bf16 matrices are row-major with the contraction dimension contiguous: a weight of a layer that
 *     maps in -> out is stored [out, in].
 *   * Confidence comparisons are taken on the canonical fixed-point softmax denominator S_q (Q28, see
 *     sfs_row_stats), never on a floating-point probability, so results do not depend on reduction order.
 */
#ifndef SFS_H_
#define SFS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SFS_OK                 0
#define SFS_ERR_INVALID_ARG   -1   /* null / misaligned pointer, size out of range, inconsistent shapes */
#define SFS_ERR_UNSUPPORTED   -2   /* a shape this build has no kernel for */
#define SFS_ERR_CUDA          -3   /* a CUDA runtime or driver call failed */
#define SFS_ERR_OOM           -4   /* workspace allocation failed */
#define SFS_ERR_STEP_LIMIT    -5   /* a sequence still had masked positions when its step budget ran out */
#define SFS_ERR_TIMEOUT       -6   /* a bounded device-side wait gave up */
#define SFS_ERR_MISSING_ROW   -7   /* the selection rule needed the statistics of a row that was not supplied */

#define SFS_LOGITS_BF16 0
#define SFS_LOGITS_F32  1

#define SFS_PHASE_SLOW 0           /* exploratory stage (Section 3.3, stage 1) */
#define SFS_PHASE_FAST 1           /* accelerated decoding stage (Section 3.3, stage 2) */

#define SFS_SAMPLER_SLOWFAST       0
#define SFS_SAMPLER_LOW_CONFIDENCE 1
#define SFS_SAMPLER_RANDOM         2

#define SFS_CONF_QBITS 28          /* S_q = sum_v trunc(2^28 * exp(x_v - max x)) */
#define SFS_MAX_W_HIST 8
#define SFS_TRACE_INTS 8

typedef struct sfs_model   sfs_model;     /* weights + shapes (borrowed device pointers) */
typedef struct sfs_session sfs_session;   /* workspace for up to max_batch x max_seq tokens; one per host thread */

/* Shape of the mask predictor (a pre-norm bidirectional transformer with RoPE, SwiGLU and RMSNorm). */
typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab, mask_id;
    float   rms_eps, rope_theta, logit_scale;
} sfs_config;

/* Device pointers to bf16 weights.  The per-layer members are HOST arrays of n_layers device pointers.
 * Everything is borrowed: it must stay valid and unchanged for the life of the model. */
typedef struct {
    const void *tok_emb;      /* [vocab, d_model] */
    const void *final_norm;   /* [d_model] */
    const void *lm_head;      /* [vocab, d_model] */
    const void *const *attn_norm;  /* [d_model] */
    const void *const *wq, *const *wk, *const *wv, *const *wo;   /* [d_model, d_model] */
    const void *const *mlp_norm;   /* [d_model] */
    const void *const *w_gate, *const *w_up;   /* [d_ff, d_model] */
    const void *const *w_down;                 /* [d_model, d_ff] */
} sfs_weights;

/* Hyper-parameters of the SlowFast rule (Section 3.3; defaults of Section 4.2 in comments). */
typedef struct {
    float   tau_min_conf;     /* 0.1   end-point threshold */
    float   tau_high_conf;    /* 0.85  parallel-unmask threshold */
    float   sigma2_stable;    /* 1.0   variance threshold of the stability check */
    int32_t k_max;            /* 8     maximum exploratory steps per cycle */
    int32_t w_hist;           /* 2     history window, 1..SFS_MAX_W_HIST */
    int32_t k_slow;           /* 1     tokens unmasked per exploratory step */
    int32_t k_fast;           /* 1     tokens unmasked by the fallback of an accelerated step */
    int32_t max_steps;        /* N; 0 means N = gen_len */
    int32_t min_high_count;   /* 1     fallback when fewer positions than this exceed tau_high_conf */
    /* The transition rule S of Eq. 4.  0 is the SlowFast rule; 1 and 2 are the LLaDA strategies of Section 3.1 that the
     * paper's tables use as the 1.00x baseline, on the same engine.  With N = max_steps (0: N = gen_len) and k = N .. 1:
     *   1 low-confidence remasking: after step k, floor(L_b * (1 - (k_b - 1) / N_b)) positions of the current block are
     *     unmasked, the most confident first (smaller S_q, ties to the lower position);
     *   2 random remasking: every masked position of the current block is unmasked with probability 1 / k_b, drawn from
     *     Philox-4x32-10 with key = seed, counter = (response position, step index N - k, sequence index, 0): unmask iff
     *     first output word * k_b < 2^32.
     * block_len cuts the response into blocks decoded left to right (semi-autoregressive remasking): block j is
     * [j * block_len, min(L, (j + 1) * block_len)), gets N / n_blocks steps (N must be a multiple of n_blocks), and L_b,
     * N_b, k_b are the block's own length, step count and countdown.  block_len 0 (or >= gen_len) is one block.
     * The SlowFast hyper-parameters above are ignored by samplers 1 and 2.  Their d_trace record is
     * (block, block start, block end, k_b, 0, n_sel, n_masked_after, k_remaining_after). */
    int32_t sampler;          /* 0 */
    int32_t block_len;        /* 0 */
    uint32_t seed_lo, seed_hi;/* 0     64-bit seed of random remasking */
} sfs_params;

/* Per-sequence scheduler state, device-resident, plain data (Algorithm 1's k, s_cycle, e_cycle, H_W, step_count). */
typedef struct {
    int32_t phase;            /* SFS_PHASE_* of the NEXT step */
    int32_t s_cycle;          /* start of the current cycle (response position) */
    int32_t hi;               /* e_cycle + 1: end of the span, meaningful in the fast phase */
    int32_t step_count;       /* exploratory steps taken in this cycle */
    int32_t hist_len;
    int32_t hist[SFS_MAX_W_HIST];   /* last e_cand values, oldest first */
    int32_t k_remaining;      /* steps still permitted */
    int32_t n_masked;
    int32_t steps_done, n_slow, n_fast, n_cycles, n_fallback;
    int32_t done;             /* 1 when no masked position is left (or the budget is spent) */
    int32_t status;           /* SFS_OK or a SFS_ERR_* detected on the device */
    int32_t reserved[10];
} sfs_state;                  /* 32 int32 = 128 bytes */

/* ---- model and session ------------------------------------------------------------------------------ */

/* Section 3.1 (the mask predictor p_theta).  Checks shapes (head_dim 64 or 128, n_heads*head_dim == d_model,
 * d_model and d_ff multiples of 8, vocab a multiple of 8), copies the pointer tables and precomputes the
 * RoPE table.  Allocates device memory; synchronises the device, so whatever wrote the weights has finished.
 * The weight arrays stay the caller's: they must outlive the model and must not be written while a call that
 * uses the model is in flight. */
int32_t sfs_model_create(const sfs_config *cfg, const sfs_weights *weights, sfs_model **out);
int32_t sfs_model_destroy(sfs_model *model);

/* Allocates every buffer a forward / generate call over at most max_batch sequences of at most max_seq
 * tokens needs (activations, logits [max_batch*max_seq, vocab] bf16, row statistics, scheduler scratch). */
int32_t sfs_session_create(sfs_model *model, int32_t max_batch, int32_t max_seq, sfs_session **out);
/* A session that can only run sfs_select (no model, hence no forward pass): allocates the selection
 * scratch for max_batch x max_seq token positions and logits rows of `vocab` entries. */
int32_t sfs_select_session_create(int32_t vocab, int32_t max_batch, int32_t max_seq, sfs_session **out);
int32_t sfs_session_destroy(sfs_session *session);

/* ---- the steps of one denoising iteration ----------------------------------------------------------- */

/* Eq. 2: logits of the mask predictor for the listed rows.
 *   d_tokens [B, S] int32.  There is no separate mask argument: the predictor's input IS the token sequence, in which
 *   a masked position holds the [MASK] token's id (Section 3.1: y^(k) is a sequence over the vocabulary that contains
 *   [MASK]); which positions are masked matters only to sfs_select, which takes the mask array.  d_rows [>= n_rows] flat token indices, or
 *   NULL for all B*S rows in order; n_rows is read from the device scalar d_n_rows when it is not NULL
 *   (then max_rows bounds it and sizes the launch), else it is max_rows.
 *   d_logits [max_rows, vocab] row-major, bf16 or fp32 per logits_dtype; row r belongs to d_rows[r]. */
int32_t sfs_forward(sfs_session *session, const int32_t *d_tokens, int32_t B, int32_t S,
                    const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                    void *d_logits, int32_t logits_dtype, void *stream);

/* Eq. 3 and the confidence equation of Section 3.1, per logits row:
 *   argmax (lowest id among equal maxima), and S_q, the fixed-point softmax denominator
 *       d = x_v - m;  r = fma(d, log2 e, 1.5*2^23);  n = r - 1.5*2^23;  f = fma(n, -ln 2, d);
 *       P = 3 + f(C1 + f(C2 + f(C3 + f C4)));  e_v = ((bits(P) << 9) mod 2^32) >> (3 - n);  S_q = sum e_v
 *   (fp32, each operation rounded once), so the confidence is c = 2^28 / S_q up to 1e-5 relative.
 *   d_logits [n_rows, ld] (ld >= vocab elements between rows).  Outputs, each optional (NULL to skip):
 *   d_argmax int32 [n_rows], d_sq uint64 [n_rows], d_conf float [n_rows] (= 2^28 / S_q, informational).
 *   n_rows comes from d_n_rows when not NULL (bounded by max_rows).  Finite or -inf logits only. */
int32_t sfs_row_stats(const void *d_logits, int32_t logits_dtype, int32_t vocab, int64_t ld,
                      const int32_t *d_n_rows, int32_t max_rows,
                      int32_t *d_argmax, uint64_t *d_sq, float *d_conf, void *stream);

/* The first of the two passes sfs_select runs over long bf16 rows (65536 to 163840 entries; other shapes return
 * SFS_ERR_UNSUPPORTED here and take the all-canonical kernels inside sfs_select): exact argmax, and an enclosure
 * d_lo[r] <= S_q <= d_hi[r] of the canonical denominator from a cheap pass (special-function exponentials, fp32 sums;
 * relative width 1.2e-4 plus vocab + 2).  sfs_select recomputes the canonical S_q only for rows whose enclosure leaves a
 * threshold comparison or the top-1 ranking of the step open, so its decisions are those of all-canonical values.
 * Exposed for tests and measurements. */
int32_t sfs_row_stats_bounds(const void *d_logits, int32_t vocab, int64_t ld, const int32_t *d_n_rows, int32_t max_rows,
                             uint64_t *d_lo, uint64_t *d_hi, int32_t *d_argmax, void *stream);

/* Initial scheduler state for B sequences of gen_len masked positions (Algorithm 1, initialisation). */
int32_t sfs_state_init(sfs_state *d_state, int32_t B, int32_t gen_len, const sfs_params *params, void *stream);

/* Section 3.3 / Algorithm 1, one step of the transition rule S for B independent sequences:
 * row statistics of the supplied logits, then per sequence the exploratory rule (top-k_slow unmasking,
 * end point e_cand, history, variance test) or the accelerated rule (unmask every in-span position above
 * tau_high_conf, else top-k_fast), the last-step rule (k == 1: unmask everything), and the phase / span
 * bookkeeping.  Updates d_tokens, d_mask and d_state in place.
 *   d_logits [n_rows, ld]; d_rows [n_rows] flat token indices b*S + pos the logits rows belong to; a
 *   sequence's step needs the rows of its masked positions in [s_cycle, L) (slow), [s_cycle, hi) (fast) or
 *   all of them (k_remaining == 1); extra rows are ignored, a missing one sets state.status =
 *   SFS_ERR_MISSING_ROW and leaves the sequence untouched.  A row index outside [0, B*S) is skipped (nothing is
 *   written for it) and reported as SFS_ERR_INVALID_ARG by sfs_check_device_status.
 *   Outputs: d_sel_count [B], d_sel_pos / d_sel_tok [B, L] (response positions ascending, and their tokens);
 *   optional d_next_rows [B*L] + d_next_n_rows [1]: the rows the following step will need, sequence-major;
 *   optional d_trace [B, SFS_TRACE_INTS]: (phase, s_cycle, hi, e_cand, stable, n_sel, n_masked_after,
 *   k_remaining_after) of this step. */
int32_t sfs_select(sfs_session *session, const void *d_logits, int32_t logits_dtype, int64_t ld,
                   const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                   int32_t *d_tokens, uint8_t *d_mask, int32_t B, int32_t S, int32_t P,
                   sfs_state *d_state, const sfs_params *params,
                   int32_t *d_sel_count, int32_t *d_sel_pos, int32_t *d_sel_tok,
                   int32_t *d_next_rows, int32_t *d_next_n_rows, int32_t *d_trace, void *stream);

/* The same step as sfs_select for callers that cannot allocate device memory (code running under a CUDA-graph
 * capture or replay, serving loops that ban allocator calls, processes whose GPU memory belongs to another
 * runtime's pool): no session is needed, because the scratch lives in a fixed array inside the library image.
 * (The paper has no counterpart of this entry point; it exists for deployment only.)
 *   Arguments as sfs_select, with `vocab` given explicitly.  Limits: B <= SFS_STATIC_MAX_BATCH sequences and
 *   B*S <= SFS_STATIC_MAX_POSITIONS token positions, else SFS_ERR_UNSUPPORTED.  The array (about 260 KB) is held
 *   by every GPU that loads the library until the process exits.  The call itself performs no cudaMalloc / cudaFree
 *   and calls no allocating routine.  All calls share the array: it keeps the previous call's contents (the call
 *   clears the parts that must start at zero), and calls whose kernels may overlap on the GPU race - run them one
 *   after another.  The first call on each device looks up the array's address; make it before any stream capture.
 *   Device-side conditions of the call (a row index outside [0, B*S), a bounded wait that gave up) are written to
 *   d_state[b].status of the call's sequences, since this entry has no session or status word to report them through. */
#define SFS_STATIC_MAX_POSITIONS 16384
#define SFS_STATIC_MAX_BATCH 64
int32_t sfs_select_static(int32_t vocab, const void *d_logits, int32_t logits_dtype, int64_t ld,
                          const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                          int32_t *d_tokens, uint8_t *d_mask, int32_t B, int32_t S, int32_t P,
                          sfs_state *d_state, const sfs_params *params,
                          int32_t *d_sel_count, int32_t *d_sel_pos, int32_t *d_sel_tok,
                          int32_t *d_next_rows, int32_t *d_next_n_rows, int32_t *d_trace, void *stream);

/* ---- feature cache (optional) ------------------------------------------------------------------------- */

/* The adaptive feature caching the paper's sampler integrates (Section 2.2; the (K_p, K_r) settings of Table 4).  The
 * paper gives no mechanism, so the rule is this library's reading: per layer the cache holds every position's rotated
 * key, value, and the residual increments of the attention and MLP branches.  Step t (from 0) recomputes the prompt
 * positions when t mod k_prompt == 0 and all response positions when t mod k_response == 0; otherwise, per layer, the
 * ceil(rho * gen_len) response positions whose fresh value vector is least similar (cosine) to the cached one (ties to
 * the lower position; in a fast step only positions of the span [s_cycle, hi) are candidates).  Recomputed queries attend
 * to all cached keys / values; every other position reuses its cached increments.  With k_prompt = k_response = 1 the
 * result is the uncached forward pass. */
typedef struct {
    int32_t k_prompt;       /* 100  prompt refresh interval */
    int32_t k_response;     /* 5    response refresh interval */
    double  rho;            /* 0.25 fraction of the response recomputed on the other steps: ceil(rho * gen_len) in double */
} sfs_cache_params;

/* Switches the cache on for the session (allocating per-layer caches for max_batch x max_seq tokens on the first call)
 * and restarts the step counter; params == NULL switches it off.  sfs_generate* then runs cached steps. */
int32_t sfs_cache_enable(sfs_session *session, const sfs_cache_params *params);
/* Restarts the step counter: the next step recomputes everything. */
int32_t sfs_cache_reset(sfs_session *session);
/* One cached forward step (as sfs_forward, for B sequences of P prompt + (S - P) response tokens); advances the step
 * counter.  d_state [B] (optional) tells slow from fast steps and gives the span; NULL means slow.  Optional dumps:
 * d_sets int32 [n_layers, B, n_sel] receives the recomputed token indices of every layer (n_sel as returned in *n_sel,
 * a HOST int), d_sims float [n_layers, B, S - P] the similarities (only written on adaptive steps).  Logits of response
 * rows are defined on every step; logits of PROMPT rows only on steps that refresh the prompt (t mod k_prompt == 0): on the
 * other steps nothing in the method reads the prompt rows of the residual stream, and they are not kept up to date. */
int32_t sfs_forward_cached(sfs_session *session, const int32_t *d_tokens, int32_t B, int32_t S, int32_t P,
                           const sfs_state *d_state, const int32_t *d_rows, const int32_t *d_n_rows, int32_t max_rows,
                           void *d_logits, int32_t logits_dtype, int32_t *d_sets, float *d_sims, int32_t *n_sel, void *stream);

/* Inspection of cached generation: from now on every cached step that sfs_generate_steps enqueues also writes its
 * recomputed token indices to d_sets [n_layers, B, n_sel] and, on adaptive steps, the similarities to d_sims
 * [n_layers, B, gen_len], exactly as sfs_forward_cached does (n_sel follows from the step counter: S on a step that
 * refreshes prompt and response, else (P if the prompt is refreshed) + (gen_len if the response is, else
 * ceil(rho * gen_len))).  The buffers are overwritten by every step; NULL pointers switch the dumps off. */
int32_t sfs_cache_dump(sfs_session *session, int32_t *d_sets, float *d_sims);

/* ---- the whole loop ------------------------------------------------------------------------------------ */

/* Algorithm 1 for B independent sequences with a common prompt length P and response length gen_len:
 * loads prompt || [MASK]*gen_len into the session, runs denoising steps (forward, row statistics,
 * selection, all on the device; finished sequences are skipped) until every sequence is done, and copies
 * the tokens out.  d_prompt [B, P]; d_out_tokens [B, P + gen_len]; d_state_out [B] optional;
 * d_trace [max_trace_steps, B, SFS_TRACE_INTS] optional.  Synchronises `stream` before returning and
 * reports SFS_ERR_STEP_LIMIT / a device-detected status if any sequence did not finish cleanly.
 * The three calls below split it so that a caller can run, time or checkpoint individual steps. */
int32_t sfs_generate(sfs_session *session, const int32_t *d_prompt, int32_t B, int32_t P, int32_t gen_len,
                     const sfs_params *params, int32_t *d_out_tokens, sfs_state *d_state_out,
                     int32_t *d_trace, int32_t max_trace_steps, void *stream);

int32_t sfs_generate_begin(sfs_session *session, const int32_t *d_prompt, int32_t B, int32_t P, int32_t gen_len,
                           const sfs_params *params, void *stream);
/* Enqueues up to n_steps denoising steps.  When d_logits_dump is not NULL, n_steps must be 1 and the bf16
 * logits of that step ([max rows, vocab]), its row list and row count are copied there for inspection. */
int32_t sfs_generate_steps(sfs_session *session, int32_t n_steps, int32_t *d_trace, int32_t max_trace_steps,
                           void *d_logits_dump, int32_t *d_rows_dump, int32_t *d_n_rows_dump, void *stream);
/* Synchronises; writes tokens / states; *n_active (host, optional) receives the number of unfinished sequences. */
int32_t sfs_generate_end(sfs_session *session, int32_t *d_out_tokens, sfs_state *d_state_out,
                         int32_t *n_active, int32_t *steps_enqueued, void *stream);

/* ---- instrumentation ------------------------------------------------------------------------------------ */

/* Kernel classes of one denoising step, in launch order. */
#define SFS_K_EMBED        0
#define SFS_K_RMSNORM      1
#define SFS_K_GEMM_QKV     2
#define SFS_K_ROPE         3
#define SFS_K_ATTENTION    4
#define SFS_K_GEMM_O       5
#define SFS_K_GEMM_GATE_UP 6
#define SFS_K_GEMM_DOWN    7
#define SFS_K_GEMM_LM_HEAD 8
#define SFS_K_ROW_STATS    9
#define SFS_K_SELECT       10
#define SFS_K_CACHE        11   /* similarity, row choice, gathers and scatters of the feature cache */
#define SFS_K_CLASSES      12

/* Per-kernel timing of a session's forward / generate launches.  First synchronises the device and, when the
 * output pointers (HOST arrays of SFS_K_CLASSES entries) are not NULL, reports the milliseconds and launch
 * counts gathered since the previous call, per kernel class; *total_launches (host, optional) receives the
 * number of kernels the session has launched since it was created.  Then timing is switched on or off for the
 * calls that follow: while on, every launch is bracketed by two CUDA events on its stream. */
int32_t sfs_profile(sfs_session *session, int32_t enable, float *ms_per_class, int64_t *launches_per_class,
                    int64_t *total_launches);

/* ---- building blocks exposed for tests and measurements ------------------------------------------------- */

/* C[M, N] = A[M, K] * B[N, K]^T, bf16 inputs, fp32 accumulation in tensor memory (tcgen05), output bf16
 * (out_dtype 0) or fp32 (1), row-major with leading dimensions lda, ldb, ldc in elements.  The same kernel
 * runs every projection of the forward pass.  K and the leading dimensions must be multiples of 8. */
int32_t sfs_linear(const void *d_A, int64_t lda, const void *d_B, int64_t ldb, void *d_C, int64_t ldc,
                   int32_t M, int32_t N, int32_t K, int32_t out_dtype, float scale, void *stream);

/* Bidirectional multi-head attention (the "a = softmax(q k^T / sqrt(dh)) v" of the mask predictor) over B
 * sequences of S tokens, no mask, in the layout the forward pass uses internally:
 *   d_qk  [B*S, 2*H*dh] bf16, per token q (H*dh values, RoPE applied) then k (H*dh values, RoPE applied);
 *   d_vt  [H*dh, B*S]   bf16, V transposed (feature-major);
 *   d_out [B*S, H*dh]   bf16.
 * head_dim 64 or 128; S a multiple of 8. */
int32_t sfs_attention(const void *d_qk, const void *d_vt, void *d_out, int32_t B, int32_t S,
                      int32_t n_heads, int32_t head_dim, void *stream);

/* Synchronises `stream` and returns (then clears) the sticky device status word: SFS_OK, or SFS_ERR_TIMEOUT
 * if a kernel's bounded wait gave up since the last check. */
int32_t sfs_check_device_status(void *stream);

const char *sfs_status_string(int32_t status);
const char *sfs_last_error(void);
int32_t     sfs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SFS_H_ */
