/*
 * l2pd — Learn2PD decoding of a masked-diffusion language model on one B200 GPU.
 *
 * C ABI.  Every pointer is marked host or device.  Nothing here throws, aborts or
 * traps the device: each call returns an l2pd_status, and l2pd_last_error() gives
 * a human-readable reason for the last failure on that context.
 *
 * The computation is the inference procedure of the Learn2PD paper (Algorithm 2, with the
 * end-of-text stop of Algorithm 3).  In this library's terms:
 *   state   a token row per sequence (prompt, then G generation positions that start as the mask
 *           token), the set of still-masked generation positions, the current block, and the
 *           effective length L_eff;
 *   step    one evaluation of the mask predictor M on every unfinished sequence, giving a
 *           prediction and a confidence for each position of the sequence's current block (Eq. 3-4),
 *           followed by the decision: the filter f_theta turns the block's confidences into
 *           probabilities (Section 3.2), masked positions whose probability exceeds tau are
 *           committed in place, and a block whose masks are all gone hands over to the next;
 *   cut     End-of-Text Prediction (Section 3.3): once an [EoT] token is committed, the positions
 *           after it leave the next step's input, and no block after that one is decoded.
 *
 * M is a LLaDA-style bidirectional transformer: token embedding, n_layers pre-norm
 * blocks (RMSNorm, fused QKV projection, rotary embedding on q and k with
 * half-split pairing, multi-head attention WITHOUT a causal mask, output
 * projection, RMSNorm, SwiGLU MLP), final RMSNorm and an untied LM head.
 * pre_j is the argmax of the LM-head logits (Eq. 3) and conf_j the softmax
 * probability of that argmax (Eq. 4); the logits are reduced on chip and never
 * stored unless a debug buffer is supplied.
 */
#ifndef L2PD_H
#define L2PD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct l2pd_ctx l2pd_ctx;   /* opaque; owned by the library */

typedef enum {
  L2PD_OK = 0,
  L2PD_ERR_ARG = -1,          /* null pointer, bad enum, bad flag */
  L2PD_ERR_SHAPE = -2,        /* sizes inconsistent with the configuration */
  L2PD_ERR_OOM = -3,          /* device or host allocation failed */
  L2PD_ERR_CUDA = -4,         /* a CUDA call failed; see l2pd_last_error */
  L2PD_ERR_TIMEOUT = -5,      /* a bounded device-side wait ran out */
  L2PD_ERR_TOKEN_RANGE = -6,  /* a prompt id outside [0, vocab) or equal to mask_id */
  L2PD_ERR_STATE = -7         /* call order: step before reset, step after all done */
} l2pd_status;

enum { L2PD_F32 = 0, L2PD_BF16 = 1 };

/* Model and decoding configuration (host memory, copied by l2pd_init). */
typedef struct {
  int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab;
  float   rms_eps;            /* y = x*g/sqrt(mean(x^2)+eps) */
  float   rope_theta;         /* angle of pair i at position t: t * theta^(-2i/head_dim) */
  int32_t mask_id, eot_id;
  int32_t dtype;              /* L2PD_F32: fp32 weights, CUDA-core arithmetic;
                                 L2PD_BF16: bf16 weights and activations, tcgen05 tensor cores,
                                 fp32 accumulation and fp32 residual stream */
  int32_t block_len;          /* s; the filter is Linear(s,s)+b -> ReLU -> Linear(s,s)+b
                                 (2*(s*s+s) parameters: 2,112 at s = 32, Section 4.1); s <= 64 */
  float   tau;                /* threshold on sigmoid(filter output); the paper uses 0.96 */
  int32_t use_filter;         /* 0: no position passes the threshold; every step commits only the
                                 most confident masked position (one token per step) */
  int32_t use_eotp;           /* 1: End-of-Text Prediction on */
  int32_t kv_cache_mode;      /* 0: every step recomputes all positions.
                                 1: block-level prefix cache (Section 4.3 names it; rule: the first
                                    step of a block runs all positions and stores K (rotated) and V of
                                    the positions before the block; the block's other steps compute
                                    only positions from the block start on and attend to
                                    stored ++ fresh keys).
                                 2: dual cache (same section): the first step of a block also stores K, V
                                    of the positions after the block; the block's other steps compute
                                    the block's s rows only and attend to stored prefix ++ fresh block
                                    ++ stored positions after the block (up to L_eff) */
  int32_t committed_conf_mode;/* what the filter reads at block positions already committed:
                                 0 = the model's confidence recomputed this step, 1 = 1.0 */
  int32_t max_batch;          /* most sequences a reset may start */
  int32_t max_seq;            /* largest P + G */
} l2pd_config;

/*
 * Weights: DEVICE pointers, borrowed — the caller keeps them alive and unchanged
 * until l2pd_destroy.  Matrices are row-major [out_features, in_features] in the
 * configuration's dtype (fp32 or bf16); norm gains, the bias and the filter are fp32.
 * The per-layer arrays are HOST arrays of n_layers device pointers (copied at init).
 */
typedef struct {
  const void *tok_emb;              /* [vocab, d_model] */
  const void *const *wqkv;          /* [3*n_heads*head_dim, d_model]: q rows, then k, then v */
  const void *const *wo;            /* [d_model, n_heads*head_dim] */
  const void *const *w_gate;        /* [d_ff, d_model] */
  const void *const *w_up;          /* [d_ff, d_model] */
  const void *const *w_down;        /* [d_model, d_ff] */
  const float *const *norm1;        /* [d_model] gain before attention */
  const float *const *norm2;        /* [d_model] gain before the MLP */
  const float *final_norm;          /* [d_model] */
  const void *lm_head;              /* [vocab, d_model] */
  const float *lm_head_bias;        /* [vocab] added to the logits, or NULL */
  const float *filt_w1, *filt_b1;   /* [s, s], [s]  (may be NULL when use_filter = 0) */
  const float *filt_w2, *filt_b2;   /* [s, s], [s] */
} l2pd_weights;

/*
 * Optional outputs of one denoising step.  Any pointer may be NULL.
 * Device arrays are indexed [sequence, j] with j the position inside the
 * sequence's current block (row stride s); rows of sequences that were already
 * finished before the step are left untouched.  Entries with P + b*s + j >= L_eff
 * (cut off by EoTP) are written as conf = 0, pred = -1.
 * Host arrays have one entry per sequence and are valid when the call returns
 * (the call then waits for the step to finish).
 */
typedef struct {
  float   *d_conf;        /* device [B, s]  Eq. 4 */
  int32_t *d_pred;        /* device [B, s]  Eq. 3 */
  float   *d_p;           /* device [B, s]  sigmoid(filter output) */
  uint8_t *d_unmask;      /* device [B, s]  1 where the step committed the position */
  float   *d_logits;      /* device [B, s, vocab] fp32 logits (debug; large) */
  int32_t *h_block;       /* host [B] block the step worked on */
  int32_t *h_masks_left;  /* host [B] masked positions left in that block after the step */
  int32_t *h_l_eff;       /* host [B] effective length P + e + 1 after the step (P + G if no EoT) */
  int32_t *h_done;        /* host [B] 1 once the sequence needs no further step */
  int32_t *h_forced;      /* host [B] 1 if the step used the progress fallback */
} l2pd_step_out;

/*
 * Create a context on `device`: validates the configuration, records the weight
 * pointers, allocates state, workspace and (kv_cache_mode != 0) the cache for
 * max_batch x max_seq.  Errors: L2PD_ERR_ARG / L2PD_ERR_SHAPE (d_model, d_ff,
 * n_heads*head_dim multiples of 8; head_dim 64 or 128 for bf16, even and <= 256 for
 * fp32; block_len in [1, 64]; ids inside the vocabulary), L2PD_ERR_OOM, L2PD_ERR_CUDA.
 * With out == NULL and ctx creation failing, `*out` is left NULL.
 */
l2pd_status l2pd_init(const l2pd_config *cfg, const l2pd_weights *w, int device, l2pd_ctx **out);

/*
 * Algorithm 2, state set-up: X <- concat(prompt, [MASK]^G) for B sequences.
 * d_prompts: DEVICE int32 [B, P].  G must be a multiple of block_len, B <= max_batch,
 * P >= 1, P + G <= max_seq (else L2PD_ERR_SHAPE).  Prompt ids are range-checked on the
 * device; a bad id makes this call return L2PD_ERR_TOKEN_RANGE (the call synchronises).
 * `stream` is a cudaStream_t (NULL = default stream).
 */
l2pd_status l2pd_state_reset(l2pd_ctx *ctx, void *stream, const int32_t *d_prompts,
                             int32_t B, int32_t P, int32_t G);

/*
 * One iteration of the while loop of Algorithm 2 for every unfinished sequence:
 * transformer forward, confidence and argmax (Eq. 3-4), filter, threshold, in-place
 * commit, EoTP, block advance.  Returns after the step's small result record has
 * reached the host (one stream synchronisation per step).  L2PD_ERR_STATE if no
 * sequence is unfinished.  `out` may be NULL.
 */
l2pd_status l2pd_denoise_step(l2pd_ctx *ctx, void *stream, const l2pd_step_out *out);

/*
 * Whole decode: l2pd_state_reset followed by l2pd_denoise_step until every sequence
 * is done.  d_out_tokens: DEVICE int32 [B, G], the response; positions after a
 * sequence's [EoT] hold eot_id.  h_out_len (HOST [B], may be NULL): tokens up to and
 * including [EoT], or G.  h_steps (HOST [B], may be NULL): number of M(X) evaluations
 * the sequence took part in.  h_total_steps (HOST, may be NULL): steps launched.
 */
l2pd_status l2pd_decode(l2pd_ctx *ctx, void *stream, const int32_t *d_prompts,
                        int32_t B, int32_t P, int32_t G, int32_t *d_out_tokens,
                        int32_t *h_out_len, int32_t *h_steps, int32_t *h_total_steps);

/*
 * Comparison policies of Section 3.1: which test a masked position of the current block must
 * pass to be committed.  The rest of the step (forward pass, confidence, progress fallback,
 * EoTP, block advance) is unchanged.
 *   L2PD_RULE_FILTER      Algorithm 2: sigmoid(filter output) > tau (the state after l2pd_init).
 *   L2PD_RULE_CONFIDENCE  confidence (Eq. 4) > conf_threshold, strict, conf_threshold in [0, 1];
 *                         at 1 nothing passes and every step commits only the most confident masked
 *                         position: the one-token-per-step decoding the paper counts speed-ups against.
 *   L2PD_RULE_EGP         Extremely Greedy Parallel: prediction == reference token.  d_reference:
 *                         DEVICE int32 [ref_rows, ref_len], borrowed until the rule is set again or the
 *                         context is destroyed; sequence i of a reset reads row i, so a reset needs
 *                         B <= ref_rows and G == ref_len (else L2PD_ERR_SHAPE).  The ids are
 *                         range-checked here (L2PD_ERR_TOKEN_RANGE; the call synchronises).  A step in
 *                         which no masked position matches commits the most confident masked position
 *                         WITH ITS REFERENCE TOKEN, so the decode ends and returns the reference.
 * The filter output p is reported as 0 under the last two rules.  Any decode in progress is
 * dropped: call l2pd_state_reset (or l2pd_decode) next.  Unused arguments are ignored.
 */
enum { L2PD_RULE_FILTER = 0, L2PD_RULE_CONFIDENCE = 1, L2PD_RULE_EGP = 2 };
l2pd_status l2pd_set_unmask_rule(l2pd_ctx *ctx, void *stream, int32_t rule, float conf_threshold,
                                 const int32_t *d_reference, int32_t ref_rows, int32_t ref_len);

/*
 * Filter depth (Section 4.4 compares one, two and four layers): replaces the two-layer filter given at
 * init by n_layers Linear(s, s) layers, z = W_n relu(... relu(W_1 c + b_1) ...) + b_n, ReLU between
 * consecutive layers, none after the last; p = sigmoid(z).  d_w, d_b: HOST arrays of n_layers DEVICE
 * pointers ([s, s] row-major and [s], fp32), borrowed until replaced or the context is destroyed.
 * n_layers = 0 goes back to the init-time filter; n_layers in [1, 4] also turns the filter on if the
 * configuration had use_filter = 0.  May be called between steps.
 */
l2pd_status l2pd_set_filter(l2pd_ctx *ctx, int32_t n_layers, const float *const *d_w, const float *const *d_b);

/*
 * Algorithm 1, stage 1 (data collection): while a sink is set, every denoising step appends one
 * sample per sequence taking part in it, in step order and, within a step, in sequence order:
 *   d_c [capacity, s] float  the filter's input of that step (the block's confidences as f_theta reads them)
 *   d_y [capacity, s] uint8  the target y_j = 1 where the prediction equals the reference token (rule
 *                            L2PD_RULE_EGP; 0 everywhere under the other rules and at positions cut off by EoTP)
 * DEVICE arrays, borrowed until the sink is replaced or cleared (NULL, NULL, 0).  A step that would
 * overflow the capacity returns L2PD_ERR_SHAPE and appends nothing.  Setting a sink resets the count.
 */
l2pd_status l2pd_set_collect(l2pd_ctx *ctx, float *d_c, uint8_t *d_y, int64_t capacity);
int64_t l2pd_collect_count(const l2pd_ctx *ctx);

/*
 * Algorithm 1, stage 2 (Eq. 6; Section 4.1): trains the two-layer filter z = W2 relu(W1 c + b1) + b2 on N
 * samples with AdamW (decoupled weight decay, bias-corrected moments, moments start at zero).  An epoch
 * visits the samples in order in batches of batch_size (0 = all N in one batch); the loss of a batch is the
 * mean over its samples and the s positions.  Arithmetic is fp32; a run is bit-reproducible on a given GPU.
 * d_c [N, s] float, d_y [N, s] uint8 (0 / 1): DEVICE.  d_w1 [s, s], d_b1 [s], d_w2 [s, s], d_b2 [s]: DEVICE fp32,
 * initial values in, trained values out.  h_losses: HOST [epochs * ceil(N / batch)] or NULL, the loss of every
 * update's batch measured before the update.  Runs on the current device, allocates and frees its scratch,
 * returns after the stream has finished.  s in [1, 64] (else L2PD_ERR_SHAPE); bad hyper-parameters L2PD_ERR_ARG.
 */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;   /* the paper gives lr = 0.001; AdamW's published defaults: 0.9, 0.999, 1e-8, 0.01 */
  int32_t epochs;                              /* the paper trains for 5,000 */
  int32_t batch_size;                          /* 0: full batch */
} l2pd_train_config;
l2pd_status l2pd_filter_train(void *stream, int32_t s, int64_t N, const float *d_c, const uint8_t *d_y, float *d_w1,
                              float *d_b1, float *d_w2, float *d_b2, const l2pd_train_config *cfg, float *h_losses);
/* The same for the depth variants of Section 4.4: n_layers in [1, 4] Linear(s, s) layers with ReLU between
 * consecutive layers.  d_w, d_b: HOST arrays of n_layers DEVICE pointers ([s, s] row-major, [s]; fp32), initial values
 * in, trained values out.  n_layers outside [1, 4] or a null entry: L2PD_ERR_ARG. */
l2pd_status l2pd_filter_train_layers(void *stream, int32_t s, int32_t n_layers, int64_t N, const float *d_c,
                                     const uint8_t *d_y, float *const *d_w, float *const *d_b,
                                     const l2pd_train_config *cfg, float *h_losses);

/* Number of sequences that still need steps (0 before the first reset). */
int32_t l2pd_num_active(const l2pd_ctx *ctx);

/* DEVICE view of the token state, int32 [B, P + G] (row stride P + G); valid until the next reset. */
const int32_t *l2pd_state_tokens(const l2pd_ctx *ctx);
/* DEVICE view of the mask set, uint8 [B, G]: 1 while the generation position is masked. */
const uint8_t *l2pd_state_masked(const l2pd_ctx *ctx);

/*
 * Debug capture (tests): when d_resid is non-NULL every following step copies the
 * fp32 residual stream into it — slot 0 after the embedding, slot l+1 after layer l —
 * as [n_layers + 1, T, d_model] with T the number of rows the step processed
 * (the caller sizes it for max_batch * max_seq rows per slot; slot stride = rows*d_model
 * where rows is the value returned through l2pd_last_step_rows).  NULL turns it off.
 */
l2pd_status l2pd_set_capture(l2pd_ctx *ctx, float *d_resid, int64_t slot_stride_elems);
int32_t l2pd_last_step_rows(const l2pd_ctx *ctx);

/* Kernels launched by this context since creation (for launch accounting). */
int64_t l2pd_launch_count(const l2pd_ctx *ctx);

/*
 * Per-kernel timing.  Kinds of kernels a step launches: */
enum {
  L2PD_K_EMBED = 0,       /* embedding gather + first RMSNorm */
  L2PD_K_GEMM_QKV = 1,    /* fused QKV projection */
  L2PD_K_ROPE = 2,        /* rotary embedding + K/V scatter */
  L2PD_K_ATTENTION = 3,   /* bidirectional attention */
  L2PD_K_GEMM_O = 4,      /* output projection + residual */
  L2PD_K_RMSNORM = 5,     /* RMSNorm */
  L2PD_K_GEMM_GATE_UP = 6,/* gate/up projection + SwiGLU */
  L2PD_K_GEMM_DOWN = 7,   /* down projection + residual */
  L2PD_K_FINAL_NORM = 8,  /* block-row gather + final RMSNorm */
  L2PD_K_LM_HEAD = 9,     /* LM head + confidence/argmax reduction */
  L2PD_K_DECIDE = 10,     /* filter, threshold, commit, EoTP */
  L2PD_K_OTHER = 11,
  L2PD_K_CHAIN = 12,      /* chained launch: O projection, RMSNorm, gate/up, down, next layer's RMSNorm and QKV */
  L2PD_K_COUNT = 13
};
/* Selects kinds (bit k = kind k) whose launches are bracketed by CUDA events on the step's
 * stream from now on, and clears the accumulated totals; mask 0 turns timing off. */
l2pd_status l2pd_profile_enable(l2pd_ctx *ctx, uint32_t kind_mask);
/* Accumulated device time (ms) and launch count of one kind since the last enable. */
l2pd_status l2pd_profile_read(const l2pd_ctx *ctx, int32_t kind, double *ms_total, int64_t *launches);

/*
 * Chained launches.  A step whose projections all run on SM pairs (bf16; up to 1536 rows) can run, per layer, the
 * attention kernel (preceded by the rotation / scatter kernel in the key/value-cache configurations) and ONE persistent
 * launch that holds the output projection, the RMSNorm before the MLP, the gate/up and down projections and the next
 * layer's RMSNorm and QKV projection: the weight loads of a projection then start while the one before it is still
 * draining, which is what the small steps of the dual cache (a few dozen rows, bound by weight streaming) gain from.
 * l2pd_set_chain(ctx, mode): 0 (the state after l2pd_init) one launch per projection; 1 chained launches where the step's
 * shapes allow, one launch per projection elsewhere; 2 the chained form's tiling in single launches (for comparisons:
 * modes 1 and 2 give bit-identical results).  With more than 256 rows the tiling does not depend on the mode, and all
 * three modes agree bit for bit; with at most 256 rows modes 1 and 2 use one 256-row slab per unit with the two
 * MMA-issuing threads on alternate k-blocks (key/value-cache configurations only).  May be called between steps.
 * Measured at 512 rows the chained and the single-launch form take the same time within a few percent (programmatic
 * dependent launch already hides the launch and the ring fill of a projection behind the one before it).
 * l2pd_chain_trace_enable(ctx, 1) makes every chained launch of the following steps record, per phase and CTA,
 * the nanosecond timer at which the CTA opened the phase, had its first and its last accumulator ready (for an
 * RMSNorm phase both equal the opening) and finished the phase; l2pd_chain_trace_read copies the last step's
 * records to HOST memory as [launch][phase slot][opened, first ready, last ready, finished][CTA] uint64 (phase
 * slots beyond a launch's phases hold stale values) and returns their count (call with h_out = NULL to size
 * the buffer; -1 on a CUDA error); it synchronises the device.  (0) frees the record buffer.
 */
l2pd_status l2pd_set_chain(l2pd_ctx *ctx, int32_t mode);
l2pd_status l2pd_chain_trace_enable(l2pd_ctx *ctx, int32_t enable);
int64_t l2pd_chain_trace_read(l2pd_ctx *ctx, uint64_t *h_out, int64_t capacity, int32_t *launches, int32_t *phases,
                              int32_t *ctas);

/*
 * Test hook for the error path: writes `code` into the context's device status word, as a kernel whose bounded
 * wait ran out would (no kernel is made to wait).  The next l2pd_denoise_step then returns L2PD_ERR_TIMEOUT and
 * clears the word; the context stays usable.  code = 0 clears it.
 */
l2pd_status l2pd_debug_set_device_status(l2pd_ctx *ctx, void *stream, int32_t code);

/* Device time of the most recent step in milliseconds (CUDA events on the step's stream),
 * or a negative value if no step has run. */
float l2pd_last_step_ms(const l2pd_ctx *ctx);

const char *l2pd_last_error(const l2pd_ctx *ctx);   /* never NULL; "" when there is none; ctx = NULL: what failed in
                                                        the calling thread's last context-free call (GEMM, LM head, ...) */
void l2pd_destroy(l2pd_ctx *ctx);                   /* NULL is allowed */

/*
 * Stand-alone kernels of the step, exported for kernel-level tests and timing.
 * All pointers are DEVICE pointers; `stream` is a cudaStream_t.  Each returns
 * L2PD_ERR_SHAPE for sizes the kernel does not support and L2PD_ERR_CUDA when the
 * launch fails; L2PD_ERR_TIMEOUT if a bounded on-device wait ran out (the call then
 * synchronises the stream to read the flag only when `check` is non-zero).
 */

/* C[M,N] (bf16) = A[M,K] (bf16, row-major) x W[N,K]^T (bf16, row-major); tcgen05 path.
 * K and N multiples of 8.  tile_n = width + 1000 * cta_group + 10000 * k_splits + 100000 * slabs
 * + 1000000 * k_interleave, every part optional (0 = chosen automatically): width a multiple of 16 in
 * [32, 256]; cta_group 1, or 2 for a pair of SMs on one 256-row tile; k_splits (residual epilogue only)
 * slices K, the slices adding into X with floating-point reductions whose order is not fixed; slabs 2
 * (pairs only) lets one unit cover two 256-row slabs against one load of the weight tile; k_interleave
 * 1 (one slab only) has two threads issue the MMAs of alternate k-blocks into two accumulators that the
 * epilogue adds (chosen automatically when the rows fit one slab), 2 switches it off.
 * A and the output follow stream order.  The weights W are requested before the kernel launched
 * just ahead of this one in the stream has completed (programmatic dependent launch): that kernel
 * must not be the one that writes them. */
l2pd_status l2pd_gemm_bf16(void *stream, const void *A, const void *W, void *C,
                           int32_t M, int32_t N, int32_t K, int32_t tile_n, int32_t check);
/* X[M,N] (fp32) += A[M,K] x W[N,K]^T : projection with the residual add in the epilogue. */
l2pd_status l2pd_gemm_bf16_residual(void *stream, const void *A, const void *W, float *X,
                                    int32_t M, int32_t N, int32_t K, int32_t tile_n, int32_t check);
/* H[M,F] (bf16) = silu(A Wg^T) * (A Wu^T), Wg and Wu [F,K] : gate/up projection with SwiGLU. */
l2pd_status l2pd_gemm_bf16_swiglu(void *stream, const void *A, const void *Wg, const void *Wu,
                                  void *H, int32_t M, int32_t F, int32_t K, int32_t tile_n,
                                  int32_t check);
/* LM head with the confidence head fused (Eq. 3-4): for each of R rows of A[R,K] (bf16),
 * pred = argmax_v (A W^T + bias)_v (lowest id on ties), conf = softmax probability of pred.
 * W [V,K] bf16, bias [V] fp32 or NULL.  d_logits (fp32 [R,V]) may be NULL.
 * d_scratch: fp32 workspace of at least l2pd_lm_head_scratch_elems(R, V) elements. */
l2pd_status l2pd_lm_head_bf16(void *stream, const void *A, const void *W, const float *bias,
                              int32_t R, int32_t V, int32_t K, float *d_scratch,
                              int32_t *d_pred, float *d_conf, float *d_logits, int32_t check);
int64_t l2pd_lm_head_scratch_elems(int32_t R, int32_t V);

/*
 * The same LM head + confidence head for callers that cannot allocate device memory.  (The paper
 * has no counterpart to this entry point; it exists for deployment reasons only.)  Some hosts run
 * this library where cudaMalloc is off limits at call time: inside a serving loop whose memory is
 * carved up front and handed out by the host's own arena, under a framework that forbids driver
 * allocations once a stream is being captured, or in a process whose device memory is fully
 * committed to weights and caches.  Those callers still pass inputs (A, W, bias) and outputs
 * (d_pred, d_conf) as DEVICE pointers, but no scratch: the per-tile reduction records go to a
 * fixed 3 MiB array compiled into the library, which every GPU that loads the library holds until
 * the process exits.  Limits: R <= 128 rows, V <= 131072; larger sizes return L2PD_ERR_SHAPE and
 * launch nothing.  The call makes no cudaMalloc/cudaFree and calls no allocating routine.
 * The first call on each device looks up the array's device address (the calling thread's current
 * device must be the one the pointers belong to); make that first call before any stream capture.
 * All calls on a device share the one array and its contents persist between calls: the call
 * clears the status word it needs at zero and rewrites every record it later reads, so stale
 * contents are harmless, but two calls that overlap on the GPU (different streams, or threads)
 * race on it — serialise them.  Results equal l2pd_lm_head_bf16's.
 */
l2pd_status l2pd_lm_head_bf16_static(void *stream, const void *A, const void *W, const float *bias,
                                     int32_t R, int32_t V, int32_t K, int32_t *d_pred, float *d_conf,
                                     int32_t check);

/* Bidirectional attention, bf16 (the mask predictor of Section 3.1 attends over the whole
 * sequence: no causal mask): q [Tq, H*dh], k and v [Tk, H*dh] (row stride given in elements),
 * out [Tq, H*dh]; softmax(q k^T / sqrt(dh)) v per head. dh 64 or 128.  All pointers are device
 * memory owned by the caller and 16-byte aligned.  impl: 0 = tensor-memory kernel (tcgen05) when
 * dh is 128 and the strides are multiples of 8, else the warp-level kernel; 1 = always the
 * warp-level (mma.sync) kernel.  check != 0 synchronises the stream and turns a device wait that
 * ran out into L2PD_ERR_TIMEOUT. */
l2pd_status l2pd_attention_bf16(void *stream, const void *q, const void *k, const void *v,
                                void *out, int32_t Tq, int32_t Tk, int32_t H, int32_t dh,
                                int64_t q_stride, int64_t kv_stride, int64_t out_stride,
                                int32_t impl, int32_t check);

/*
 * Environment switches (read once, at l2pd_init or at the first call that uses them; diagnostics and
 * comparisons only — the defaults are the product):
 *   L2PD_FORCE_SIMT=1       bf16 configurations run their GEMMs and attention on the CUDA-core cross-check kernels
 *   L2PD_ATTN_WARP=1        head size 128 keeps the warp-level (mma.sync) attention kernel instead of tcgen05
 *   L2PD_NO_ROPE_FUSION=1   rotary embedding as a separate kernel instead of the QKV epilogue
 *   L2PD_NO_PDL=1           kernels launched without programmatic dependent launch
 *   L2PD_ATOMIC_KSPLIT=1    K slices of the O / down projections add into x in completion order (not
 *                           bit-reproducible) instead of storing partial sums that are added in slice order
 *   L2PD_DIRECT_STORES=1    stand-alone GEMM calls use per-thread stores in the epilogue instead of staged TMA stores
 */

#ifdef __cplusplus
}
#endif
#endif /* L2PD_H */
