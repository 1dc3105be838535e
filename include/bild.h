/* libbild: the batch-1 decode loop of Big Little Decoder (BiLD) for one pair of
 * T5-shaped encoder-decoder models on one GPU (sm_100a).
 *
 * What the calls compute is defined by the paper:
 *   - problem statement, Section 3.2 (Eq. 1-2): at every step the next token comes
 *     from the small or from the large model, chosen by a boolean policy;
 *   - fallback policy, Section 3.3: hand over to the large model when the small
 *     model's largest softmax probability is below alpha_FB;
 *   - rollback policy, Section 3.4 (Eq. 3): the large model reads all pending
 *     small-model tokens in ONE non-autoregressive pass; the first position whose
 *     distance d = -ln p_L(small model's token) exceeds alpha_RB is replaced by
 *     the large model's token and everything after it is dropped;
 *   - the whole loop, Algorithm 1 (Section 3.5);
 *   - d is the cross entropy between the small model's hard label and the large
 *     model's soft label (Section 4.1), and the small model writes at most
 *     `max_draft` tokens in a row (evaluation details, supplementary material).
 * The paper names its models (T5 / mT5, Section 4.1 and the model-size table)
 * but does not define them; the architecture implemented is stated at
 * bild_model_cfg below.
 *
 * General rules
 *   - Every pointer is tagged HOST or DEVICE.  The library never allocates or
 *     frees device memory: weights, workspace and debug buffers are the caller's
 *     and must outlive the context.  bild_create allocates a small host-side
 *     context, freed by bild_destroy.
 *   - Every call returns a status (BILD_OK = 0 or a negative BILD_ERR_*), never
 *     throws, never aborts.  After an error the context is usable again after
 *     bild_encode.  bild_last_error gives a message for the last failing call.
 *   - All work is enqueued on the CUDA stream given to bild_create.  Calls that
 *     return results in host memory synchronise that stream before returning.
 *   - A context is not thread-safe; use one context per host thread.
 */
#ifndef BILD_H
#define BILD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bild_ctx bild_ctx; /* opaque */

enum {
  BILD_OK = 0,
  BILD_ERR_ARG = -1,       /* null pointer, value out of range */
  BILD_ERR_WORKSPACE = -2, /* workspace too small or misaligned */
  BILD_ERR_STATE = -3,     /* call out of order (e.g. decode before bild_encode) */
  BILD_ERR_CAPACITY = -4,  /* sequence would exceed max_enc_len / max_dec_len */
  BILD_ERR_CUDA = -5,      /* a CUDA runtime call failed */
  BILD_ERR_TIMEOUT = -6    /* a bounded device-side wait expired */
};
enum { BILD_FP32 = 0, BILD_BF16 = 1 };              /* storage type of weight matrices */
enum { BILD_FFN_RELU = 0, BILD_FFN_GATED_GELU = 1 };
enum { BILD_MODE_BILD = 0, BILD_MODE_SMALL_ONLY = 1, BILD_MODE_LARGE_ONLY = 2 };
enum { BILD_MAX_BLOCK = 16 };                       /* largest k of bild_large_verify */

/* One encoder-decoder model.  Architecture (T5 / mT5 as published): pre-norm
 * residual blocks; RMS norm y = x*g/sqrt(mean(x^2)+ln_eps) without bias; attention
 * scores not scaled by 1/sqrt(d_kv); additive relative-position bias on
 * self-attention only, one [rel_buckets][n_heads] table per stack shared by its
 * layers (decoder: unidirectional buckets, encoder: bidirectional); cross-attention
 * without bias or mask; FFN = ReLU or tanh-GELU gate; final RMS norm;
 * logits = logit_scale * W_lm h.  Encoder and decoder have the same depth/width. */
typedef struct {
  int32_t n_layers, d_model, n_heads, d_kv, d_ff, ffn_kind, vocab;
  int32_t rel_buckets;   /* 32 */
  int32_t rel_max_dist;  /* 128 */
  float ln_eps;          /* 1e-6 */
  float logit_scale;
} bild_model_cfg;

typedef struct {
  bild_model_cfg small_cfg, large_cfg;
  int32_t dtype;        /* BILD_FP32 or BILD_BF16: type of every matrix and of the embedding table */
  int32_t max_enc_len;  /* capacity for encoder ids */
  int32_t max_dec_len;  /* capacity of y including the start symbol: max_len + 1 <= max_dec_len */
  int32_t max_draft;    /* small-model tokens in a row before a forced fallback (paper: 10); 1..15 */
  int32_t start_id;     /* y[0] */
  int32_t eos_id;       /* -1: never stop on a token */
  /* Early-exit configuration (Section 4.4, "Early Exiting Strategy"): n > 0 makes the small model the first n
   * decoder layers of the large model, with the large model's encoder, embedding, final norm and prediction
   * head.  small_cfg must then equal large_cfg except for n_layers (= n) and logit_scale; the small model's
   * weights argument is ignored (may be NULL); only the large model's encoder runs, and the two "models"
   * share the cross-attention K/V and the self-attention cache of those n layers (a large pass rewrites the
   * rows the small steps wrote, so the cache always holds the large model's own values).  0: two models. */
  int32_t early_exit_layers;
} bild_config;

/* All members are DEVICE pointers.  Matrices are row-major [out][in] in
 * config.dtype; norm gains and bias tables are always fp32.  inner = n_heads*d_kv. */
typedef struct {
  const void *ln1;   /* [d] fp32 */
  const void *wqkv;  /* [3*inner][d], rows: q, k, v */
  const void *wo;    /* [d][inner] */
  const void *ln2;   /* [d] fp32 */
  const void *wi0;   /* [d_ff][d]  (ReLU branch, or GELU branch of the gate) */
  const void *wi1;   /* [d_ff][d]  linear branch of the gate; NULL for ReLU */
  const void *wfo;   /* [d][d_ff] */
} bild_enc_layer;

typedef struct {
  const void *ln1, *wqkv, *wo;  /* self-attention, as above */
  const void *ln2;              /* [d] fp32 */
  const void *wcq;              /* [inner][d] */
  const void *wckv;             /* [2*inner][d], rows: k, v (applied to the encoder memory) */
  const void *wco;              /* [d][inner] */
  const void *ln3;              /* [d] fp32 */
  const void *wi0, *wi1, *wfo;  /* as above */
} bild_dec_layer;

typedef struct {
  const void *emb;           /* DEVICE [vocab][d] */
  const void *lm_head;       /* DEVICE [vocab][d]; may equal emb */
  const void *enc_rel_bias;  /* DEVICE [rel_buckets][n_heads] fp32 */
  const void *dec_rel_bias;  /* DEVICE [rel_buckets][n_heads] fp32 */
  const void *enc_final_ln;  /* DEVICE [d] fp32 */
  const void *dec_final_ln;  /* DEVICE [d] fp32 */
  const bild_enc_layer *enc_layers; /* HOST array [n_layers] of structs of DEVICE pointers (copied) */
  const bild_dec_layer *dec_layers; /* HOST array [n_layers] (copied) */
} bild_weights;

/* Result of one small-model step (Algorithm 1, the small-model branch). */
typedef struct {
  int32_t argmax;   /* lowest index among equal maxima */
  float max_logit;
  float lse;        /* ln sum exp of the scaled logits */
  float pmax;       /* largest softmax probability */
  int32_t fallback; /* 1 iff pmax < alpha_fb (Section 3.3) */
} bild_step_out;

/* Result of one large-model block pass (Algorithm 1, the fallback branch). */
typedef struct {
  int32_t argmax[BILD_MAX_BLOCK];  /* row i: arg max of p_L(. | y up to and including tokens[i]) */
  float lse[BILD_MAX_BLOCK];
  float d[BILD_MAX_BLOCK];         /* d[i] = -ln p_L(tokens[i+1]) under row i, i < k-1 */
  int32_t first_violation;         /* smallest i < k-1 with d[i] > alpha_rb, else -1 (Eq. 3) */
  int32_t next_token;              /* argmax[first_violation], else argmax[k-1] */
} bild_verify_out;

/* kind: 0 small token accepted (token written at y[pos], value = p_max)
 *       1 fallback, 2 forced fallback after max_draft drafts (token = the small model's
 *         rejected candidate for y[pos], value = p_max)
 *       3 large pass without rollback, 4 with rollback (token written at y[pos],
 *         k = block size, m = first violating row or -1, value = d[m], or for kind 3 the
 *         largest distance scanned, 0 if none). */
typedef struct {
  int32_t kind, pos, token, k, m;
  float value;
} bild_trace_rec;

typedef struct {
  int32_t small_steps, large_calls, fallbacks, forced, rollbacks, discarded, sum_k;
} bild_stats;

/* Bytes of DEVICE workspace bild_create needs for this configuration (KV caches,
 * cross-attention K/V, activations, kernel scratch, decode state, trace). */
int bild_query_workspace(const bild_config *cfg /*HOST*/, size_t *bytes /*HOST out*/);

/* Build a context.  `workspace` is DEVICE memory, 256-byte aligned, at least
 * bild_query_workspace bytes, caller-owned, used exclusively by this context until
 * bild_destroy.  `cuda_stream` is a cudaStream_t (NULL = default stream).  Device work done
 * here, on that stream, with a synchronisation before returning: the workspace is cleared
 * and the relative-position bias tables are expanded by distance.  The weights are read in
 * place by every kernel (no copies, no re-layout).  Errors: ARG, WORKSPACE, CUDA. */
int bild_create(const bild_config *cfg /*HOST*/, const bild_weights *small_w /*HOST*/,
                const bild_weights *large_w /*HOST*/, void *workspace /*DEVICE*/,
                size_t workspace_bytes, void *cuda_stream, bild_ctx **out /*HOST out*/);

/* Kernel selection and debugging switches (no counterpart in the paper).  The product path is
 * what bild_tuning_default() fills in and what bild_create uses; tests and measurements set
 * single fields to reach the comparison kernels.  Nothing is read from the environment. */
typedef struct {
  int32_t host_loop;         /* 1: bild_generate is driven from the host, one state read-back per pass (debug) */
  int32_t pdl;               /* 1: kernels of a pass are launched with programmatic dependent launch */
  int32_t fused;             /* fused sub-layer kernels: 0 off, 1 single-row passes, 2 also passes of 2 to 8 rows, 3 also
                              * blocks of 9 to 16 rows (as two chunks of up to 8 rows on two streams, layer l of the second
                              * chunk waiting for the self-attention of layer l of the first) */
  int32_t ffn_parts;         /* launches the fused feed-forward sub-layer is split into (0: fewest that fit) */
  int32_t block_simt;        /* 1: unfused block passes on the SIMT block GEMV */
  int32_t slice_mode;        /* unfused linear layers on the row-slice kernel: 0 off, 1 block passes, 2 also single rows */
  int32_t slice_min_kb;      /* single-row passes: matrices below this size stay on the GEMV */
  int32_t slice_mma_min;     /* row-slice kernel: row counts from this on use tensor-core tiles (2..5) */
  int32_t slice_head;        /* tensor-core LM head: 0 off, 1 block passes, 2 also single rows of large heads */
  int32_t slice_head_min_mb; /* single rows: heads from this size on */
  int32_t unit_attn;         /* 1: unfused decoder attention on the chunked 256-thread kernel */
  int32_t umma;              /* 1: tcgen05 kernels (encoder linears; unfused block linears when slice_mode = 0) */
  int32_t enc_gemm;          /* 1: encoder linears as 128-token tcgen05 GEMM tiles */
  int32_t enc_attn_mma;      /* 1: encoder self-attention on mma.sync tiles */
  int32_t enc_parallel;      /* 1: the two encoders run side by side on two streams, and the cross K/V projections of the
                              * decoder layers on three; 0: the whole set-up step on the context's stream */
  int32_t spin_limit;        /* polls before a bounded device-side wait gives up with BILD_ERR_TIMEOUT (0: 2^20) */
  int32_t debug_skip_copies; /* 1: the fused attention kernel announces its weight copies but does not issue them, so
                              * that its bounded wait runs out (test of the time-out path; never set in production) */
  int32_t attn_all_keys;     /* fused attention: while a head has at most this many keys (and they fit one staged chunk)
                              * every block of the head's cluster attends over all of them, which saves the exchange
                              * and merge of per-block partial results; 0: keys always split over the cluster */
  int32_t graph_switch;      /* 1: in the loop graph the large pass of an iteration hangs off ONE conditional node of the
                              * SWITCH kind (bodies: block pass, single-row pass, pass of 2 to 8 rows); 0: one IF node per
                              * kind of pass */
  int32_t enc_split_k;       /* 1: encoder GEMMs that add to the residual stream (output projection, second FFN matrix)
                              * split K over more blocks, partial tiles added with reductions at the L2 */
  int32_t head_stream;       /* single-row bf16 LM heads (rows of at most 1024 columns) on the streaming kernel: 0 off,
                              * 1 heads of slice_head_min_mb and more, 2 all */
  int32_t enc_attn_groups;   /* encoder self-attention (enc_attn_mma): groups of four warps per block, each visiting every
                              * n-th tile of 64 keys, partial results merged at the end; 1..3 */
} bild_tuning;
void bild_tuning_default(bild_tuning *t /*HOST out*/);
/* bild_create with explicit switches; tuning == NULL means the defaults. */
int bild_create_tuned(const bild_config *cfg, const bild_weights *small_w, const bild_weights *large_w,
                      void *workspace, size_t workspace_bytes, void *cuda_stream,
                      const bild_tuning *tuning /*HOST*/, bild_ctx **out);
void bild_destroy(bild_ctx *ctx); /* frees the host-side context only */

/* Run both encoders over ids[0..n_ids) and project the cross-attention K/V of
 * every decoder layer (the per-input set-up of Algorithm 1's two models).  Resets
 * the decode state: y = [start_id], both caches empty.  1 <= n_ids <= max_enc_len.
 * Asynchronous on the stream (ids are copied before returning).  The small model's
 * encoder runs on a stream of the context's own, forked from and joined back into the
 * caller's stream with events, so work queued on the caller's stream after this call still
 * sees both encoders' results (bild_tuning.enc_parallel = 0 keeps everything on the caller's
 * stream). */
int bild_encode(bild_ctx *ctx, const int32_t *ids /*HOST*/, int n_ids);

/* Reset the decode state only (keeps the encoder results of the last bild_encode). */
int bild_reset(bild_ctx *ctx);

/* One small-model step: feed `token` at the next position of the small model's
 * cache (cache length += 1) and return the arg-max / p_max / fallback test of the
 * next-token distribution (Section 3.3).  logits_dbg: DEVICE [vocab] fp32 or NULL;
 * when given, the scaled logits are also written there (debug; the normal path
 * never stores them).  Synchronises. */
int bild_small_step(bild_ctx *ctx, int32_t token, float alpha_fb, bild_step_out *out /*HOST*/,
                    float *logits_dbg /*DEVICE or NULL*/);

/* One large-model block pass over tokens[0..k), 1 <= k <= BILD_MAX_BLOCK, fed at the
 * next k positions of the large model's cache (cache length += k; no rewind is done
 * here).  Row i is the distribution after tokens[i]; tokens[i+1] is judged by row i
 * (Section 3.4).  logits_dbg: DEVICE [k][vocab] fp32 or NULL.  Synchronises. */
int bild_large_verify(bild_ctx *ctx, const int32_t *tokens /*HOST*/, int k, float alpha_rb,
                      bild_verify_out *out /*HOST*/, float *logits_dbg /*DEVICE or NULL*/);

/* Cut a self-attention cache back to new_len rows (which: 0 small, 1 large).  Only a
 * length counter changes; later steps overwrite the dropped rows. */
int bild_rewind(bild_ctx *ctx, int which, int new_len);

/* Algorithm 1 from y = [start_id] until max_len tokens exist or eos_id was written.
 * Resets the decode state first (bild_encode must have been called).  The loop runs
 * on the device; tokens, trace and counters are copied back once at the end.
 * tokens_out: HOST [max_len]; *n_tokens: number written.  trace_out: HOST
 * [trace_cap] or NULL; *n_trace = records produced (records beyond trace_cap are
 * counted but dropped).  mode: BILD_MODE_*.  Synchronises.
 * Errors: STATE (no encode), CAPACITY (max_len + 1 > max_dec_len), ARG, CUDA. */
int bild_generate(bild_ctx *ctx, int mode, float alpha_fb, float alpha_rb, int max_len,
                  int32_t *tokens_out /*HOST*/, int *n_tokens /*HOST out*/,
                  bild_trace_rec *trace_out /*HOST or NULL*/, int trace_cap, int *n_trace /*HOST out*/,
                  bild_stats *stats /*HOST out or NULL*/);

/* As bild_generate, but only enqueues the device loop (no copy back, no sync): for
 * timing with events on the stream.  Fetch the results with bild_fetch_result. */
int bild_generate_async(bild_ctx *ctx, int mode, float alpha_fb, float alpha_rb, int max_len);
int bild_fetch_result(bild_ctx *ctx, int32_t *tokens_out /*HOST*/, int *n_tokens /*HOST out*/,
                      bild_trace_rec *trace_out /*HOST or NULL*/, int trace_cap, int *n_trace,
                      bild_stats *stats /*HOST out or NULL*/);

/* Measurement aid for the per-pass latencies (the paper's claim under test is that one
 * block pass over k tokens costs one weight load, Section 3.2): run one decoder pass of
 * model `which` (0 small with k = 1, 1 large with 1 <= k <= 16) `iters` times back to back
 * at self-cache length cache_len, with whatever the cache holds, and return the mean time
 * of one pass in milliseconds (CUDA events on the context's stream).  One untimed pass
 * runs first; with iters < 0 it does not (|iters| timed passes), so that the first timed pass
 * finds the caches as the previous work left them ("L2-cold" step after a large pass).
 * Leaves the decode state undefined: call bild_reset or bild_generate afterwards.
 * Synchronises. */
int bild_time_pass(bild_ctx *ctx, int which, int k, int cache_len, int iters, float *ms_per_pass /*HOST out*/);

/* The sampling variant (supplementary material, section "BiLD with Sampling"): both models draw
 * their tokens by nucleus sampling with mass top_p (0 < top_p <= 1; the paper uses 0.8) instead of
 * taking the arg-max, while the fallback test (maximum probability of the small model) and the rollback
 * test (-ln p_L of the token the small model drew) stay as they are.  The random numbers are inputs:
 * u_small[j] / u_large[j] in [0, 1) is used when the small / large model draws the token written to
 * y[j], j = 1 .. max_len (HOST arrays of max_len + 1 floats; a position drawn again after a rollback
 * uses the same number).  Nucleus: tokens in order of decreasing probability (equal: lower index
 * first), shortest prefix with mass >= top_p; drawn token: first of the prefix at which the running sum
 * exceeds u times the prefix's mass.  Otherwise as bild_generate; the LM heads keep their logits in the
 * workspace in this mode and one more kernel per pass draws the token. */
int bild_generate_sampled(bild_ctx *ctx, int mode, float alpha_fb, float alpha_rb, int max_len,
                          float top_p, const float *u_small /*HOST*/, const float *u_large /*HOST*/,
                          int32_t *tokens_out /*HOST*/, int *n_tokens /*HOST out*/,
                          bild_trace_rec *trace_out /*HOST or NULL*/, int trace_cap, int *n_trace,
                          bild_stats *stats /*HOST or NULL*/);

/* 1 if the tcgen05 kernels are in use for this context (bf16 weights, d_model / inner / d_ff
 * multiples of 64): they run the ENCODER's linear layers (the set-up step) and, with
 * bild_tuning.fused = 0 and slice_mode = 0, the linear layers of block passes.  The decoder passes of
 * the product path multiply on mma.sync tiles (blocks of 2 rows and more) or plain multiply-adds
 * (single rows): they are latency-bound, see the per-pass tables.  0: no tcgen05 kernel runs. */
int bild_uses_tensor_cores(const bild_ctx *ctx);

/* Number of kernel launches this context has enqueued since it was created. */
int64_t bild_launch_count(const bild_ctx *ctx);

const char *bild_last_error(const bild_ctx *ctx); /* HOST string owned by the context */

/* ---- single operations (for unit tests and micro-benchmarks) -------------------
 * One kernel (or one sub-layer) run once on the given stream, every pointer DEVICE unless said
 * otherwise.  bild_op_linear and bild_op_lm_head run the per-operation kernels (GEMV / SIMT linear,
 * single-row and SIMT heads) that fp32 configurations and odd shapes use; bild_op_lm_head_sliced,
 * bild_op_lm_head_stream, bild_op_attn_sublayer and bild_op_ffn_sublayer run the kernels the bf16
 * decoder passes use. */

/* Y[m][n] = sum_j W[n][j] * H[m][j], H = X if gain == NULL, else the RMS norm of X
 * with that gain (Section 3.2's model forward; one weight pass serves all m rows).
 * W: [N][K] in w_dtype; X: [M][K] fp32; Y: [M][N] fp32.  1 <= M <= BILD_MAX_BLOCK. */
int bild_op_linear(const void *W, int w_dtype, const float *X, const float *gain, float eps,
                   float *Y, int M, int N, int K, void *cuda_stream);

/* Fused LM head (Sections 3.3 and 3.4): for each of M rows, z = scale * W_lm rms(X),
 * and from z only: arg-max (lowest index), max, ln-sum-exp, and z[target[m]]
 * (target may be NULL).  The logits are not stored unless logits_dbg != NULL.
 * scratch: at least bild_op_lm_head_scratch_bytes(V) bytes, 256-byte aligned.
 * K <= 4096; for M >= 2 also 16 rows of K floats must fit a block's shared memory (K up to
 * about 3500), else BILD_ERR_CAPACITY. */
size_t bild_op_lm_head_scratch_bytes(int V);
int bild_op_lm_head(const void *W, int w_dtype, const float *X, const float *gain, float eps,
                    float scale, const int32_t *target, int M, int V, int K,
                    int32_t *argmax_out, float *max_out, float *lse_out, float *gather_out,
                    float *logits_dbg, void *scratch, void *cuda_stream);

/* The same fused head on the tensor-core kernel of the bf16 decoder passes (one block per SM, the
 * vocabulary streamed through shared memory by bulk copies): W bf16 [V][K], 16-byte aligned;
 * K * (3 * tile rows * 2 + 64) bytes must fit a block (K <= 2048), else BILD_ERR_CAPACITY.
 * scratch as for bild_op_lm_head.  Asynchronous on the stream. */
int bild_op_lm_head_sliced(const void *W, const float *X, const float *gain, float eps, float scale,
                           const int32_t *target, int M, int V, int K, int32_t *argmax_out,
                           float *max_out, float *lse_out, float *gather_out, float *logits_dbg,
                           void *scratch, void *cuda_stream);

/* The same fused head for ONE row on the streaming kernel of the bf16 single-row passes (two blocks per SM walk the
 * vocabulary, weights through registers): W bf16 [V][K], 16-byte aligned, K <= 1024 (else BILD_ERR_CAPACITY), X [K].
 * scratch as for bild_op_lm_head.  Asynchronous on the stream. */
int bild_op_lm_head_stream(const void *W, const float *X, const float *gain, float eps, float scale,
                           const int32_t *target, int V, int K, int32_t *argmax_out, float *max_out,
                           float *lse_out, float *gather_out, float *logits_dbg, void *scratch,
                           void *cuda_stream);

/* One decoder sub-layer on the fused kernels of the bf16 passes (Section 3.2's model forward, one
 * weight pass for all M rows; steps S1-S3 / S4-S6 / S7-S8 of the small step, L1-L8 of the block
 * pass): x_out = x_in + SubLayer(rms_norm(x_in) * gain).  1 <= M <= 8; x_in, x_out fp32 [M][d];
 * all weights bf16, row-major [out][in], 16-byte aligned.  scratch: bild_op_sublayer_scratch_bytes(d, F)
 * bytes (F = 0 for attention), 256-byte aligned.  Both calls synchronise the stream before returning
 * and return BILD_ERR_TIMEOUT if a bounded wait inside the kernel ran out; BILD_ERR_ARG for shapes the
 * fused kernels do not take (d <= 1024, d_kv in {16, 32, 64}, ...).
 *   attention: self != 0: Wp = [3 H d_kv][d] (q, k, v rows); the M rows sit at positions n_before ..
 *     n_before + M - 1, attend causally over the n_before cached rows of kc / vc ([H][cap][d_kv] fp32)
 *     and themselves, with bias_by_dist [H][cap] added by distance; their keys / values are appended to
 *     kc / vc.  self == 0: Wp = [H d_kv][d]; the rows attend over the n_before rows of kc / vc.
 *   feed-forward: Wi0 (and the GELU gate Wi1, or NULL for ReLU) [F][d], Wfo [d][F]; `parts` = launches
 *     the slice of d_ff per block is split over (0: fewest that fit). */
size_t bild_op_sublayer_scratch_bytes(int d, int F);
int bild_op_attn_sublayer(int self, const void *Wp, const void *Wo, const float *gain, float eps,
                          const float *x_in, float *x_out, float *kc, float *vc, int cap, int n_before,
                          const float *bias_by_dist, int M, int d, int H, int dkv, void *scratch,
                          void *cuda_stream);
int bild_op_ffn_sublayer(const void *Wi0, const void *Wi1, const void *Wfo, const float *gain, float eps,
                         const float *x_in, float *x_out, int M, int d, int F, int parts, void *scratch,
                         void *cuda_stream);

/* The paper has no counterpart for this call; it exists for callers that cannot allocate.
 * Same computation and outputs as bild_op_lm_head, but the kernel's scratch (block
 * partials, ticket counter, result record) is a fixed 128 KiB array inside the library's
 * device image, so the caller passes no scratch and nothing is allocated here: no
 * cudaMalloc / cudaFree, no allocating library routine.  Meant for a decode worker inside
 * a serving process whose allocator already owns the device's memory, or for a
 * latency-critical loop where cudaMalloc's device-wide synchronisation is not acceptable.
 *   - Limits: M <= 16, V <= 1048576, K <= 4096 (multiple of 8), and for M >= 2 the kernel
 *     stages 16 rows of K floats in shared memory, which a block can hold for K up to about
 *     3500 on a B200 (the exact bound is taken from the device's attributes); beyond any of
 *     them the call returns BILD_ERR_CAPACITY (and says why on stderr).  bild_op_lm_head
 *     has no V limit of its own but the same shared-memory bound for M >= 2, with the same
 *     error.
 *   - Every GPU that loads the library holds the 128 KiB until the process exits.
 *   - The first call on a device looks the array's device address up (a runtime call that
 *     is not a stream operation), so make that first call before any stream capture, with
 *     the intended device current.
 *   - All calls on a device share the one array and it keeps the previous call's
 *     contents; the call clears what must start at zero on the given stream.  Two calls
 *     whose kernels overlap on the GPU (different streams, no ordering) race on it and
 *     give wrong results: order them.
 *   - No logits debug dump.  Asynchronous on the stream; all pointers DEVICE. */
int bild_op_lm_head_static(const void *W, int w_dtype, const float *X, const float *gain, float eps,
                           float scale, const int32_t *target, int M, int V, int K,
                           int32_t *argmax_out, float *max_out, float *lse_out, float *gather_out,
                           void *cuda_stream);

/* Test helper: one decoder layer's cached keys or values as the kernels see them, copied to
 * HOST memory (synchronises the stream).  which: 0 small, 1 large model; what: 0 cross-attention
 * keys, 1 cross-attention values (written by bild_encode: W_ck / W_cv times the encoder output,
 * the per-input set-up of Section 3.2's two models), 2 / 3 self-attention keys / values (rows
 * appended by the decoder passes).  Layout [n_heads][capacity][d_kv] fp32 with capacity =
 * max_enc_len (cross) or max_dec_len (self); count must be exactly that many floats. */
int bild_debug_read_cache(bild_ctx *ctx, int which, int what, int layer, float *dst_host, size_t count);

/* Host-only: the relative-position bucket the library uses (T5's bucket function in
 * exact integer arithmetic).  which = 0: decoder, rel = query_pos - key_pos >= 0;
 * which = 1: encoder, rel = key_pos - query_pos.  Returns -1 on invalid arguments. */
int bild_debug_bucket(int which, int rel, int n_buckets, int max_dist);

#ifdef __cplusplus
}
#endif
#endif /* BILD_H */
