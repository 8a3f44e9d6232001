/*
 * fdvlm.h -- C ABI of the B200 (sm_100a) block-diffusion denoise-step library.
 *
 * One handle = one request at batch size one of a Qwen2.5-shaped decoder run as a block-diffusion
 * language model (Fast-dVLM, Sec. 3.4 "Inference" and Appendix B, Alg. 1):
 *
 *   fdvlm_prefill       causal forward over the prefix (vision embeddings, then text tokens) that
 *                       fills the KV cache                               (Alg. 1, "Prefill")
 *   fdvlm_block_begin   start a block of B positions, all [MASK] unless tokens are given (Sec. 3.4)
 *   fdvlm_block_step    one denoise step: forward of the B block rows -- bidirectional inside the
 *                       block, full over the cache, cache NOT updated (Alg. 1 draft step; Sec. 3.3
 *                       M_N2N, M_N2C) -- then softmax max-probability confidence and
 *                       threshold / top-k parallel unmasking (Sec. 3.4; Sec. 4.5)
 *   fdvlm_commit_block  causal forward of the finished block WITH cache update (Alg. 1 verify step;
 *                       Sec. 3.3 M_C2C: clean context is token-causal)
 *
 * and, built from the same forward: the decode loops without host round trips (fdvlm_decode_block_topk,
 * fdvlm_decode_block), the commit fused into the next block's first step (fdvlm_commit_begin_step,
 * fdvlm_commit_decode_block(_topk)), linear and quadratic self-speculative decoding (fdvlm_spec_block, Alg. 1;
 * fdvlm_quad_begin / fdvlm_quad_step, Alg. 2), W8A8 (FDVLM_W8A8_FP8E4M3), and the single operators.
 *
 * Conventions
 *   - All `device` pointers are CUDA device memory of the handle's GPU; `host` pointers are ordinary
 *     host memory.  No pointer is retained beyond a call except the weight pointers given to
 *     fdvlm_create, which are BORROWED and must stay valid and unchanged until fdvlm_destroy.
 *   - Matrices are row-major [out_features, in_features] (K contiguous); vectors are dense.
 *   - The KV cache, workspace and block state belong to the handle (allocated in fdvlm_create with
 *     cudaMalloc, freed in fdvlm_destroy).
 *   - All work is issued on the CUDA stream given at create time.  Calls that return data to the host
 *     (info / *_host variants) synchronise that stream before returning; others are asynchronous.
 *   - Every function returns FDVLM_OK (0) or a negative fdvlm_status; argument and state errors are
 *     detected on the host before anything is launched.  fdvlm_last_error gives a message.
 *   - A handle is not thread-safe; distinct handles are independent.  There is no CPU fallback: with
 *     no usable GPU fdvlm_create fails with FDVLM_ERR_CUDA.
 */
#ifndef FDVLM_H_
#define FDVLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fdvlm fdvlm_t; /* opaque */

typedef enum {
  FDVLM_OK = 0,
  FDVLM_ERR_INVALID_ARG = -1, /* NULL / out-of-range argument, unsupported shape relation          */
  FDVLM_ERR_STATE = -2,       /* step without begin, commit with masks left, begin inside a block  */
  FDVLM_ERR_CAPACITY = -3,    /* cache_len + rows > max_seq, or block_size > max_block             */
  FDVLM_ERR_UNSUPPORTED = -4, /* shape or dtype the kernels do not cover                           */
  FDVLM_ERR_CUDA = -5,        /* a CUDA runtime call failed (message has the CUDA error string)    */
  FDVLM_ERR_TIMEOUT = -6,     /* a bounded device-side wait gave up; outputs of that call invalid  */
  FDVLM_ERR_OOM = -7          /* device allocation failed in fdvlm_create                          */
} fdvlm_status;

/* Storage type of the linear weights.  For FDVLM_F32 everything is fp32.  Otherwise the embedding table and the
 * embedding rows given to fdvlm_prefill are bf16, and the accumulation, residual stream, norms and softmax are
 * fp32; the 16-bit tensors between the operators are internal: GEMM inputs are pairs of bf16 (value = hi + lo, ~16
 * significant bits) for bf16 weights and f16 for fp8 weights (e4m3 widens exactly to f16), q and the KV cache are
 * of fdvlm_kv_dtype. */
typedef enum {
  FDVLM_F32 = 0,
  FDVLM_BF16 = 1,
  FDVLM_W_FP8E4M3 = 2, /* OCP e4m3fn bytes + fp32 per-output-channel scale: w = e4m3(byte) * scale[out] */
  /* W8A8 (Sec. 3.4 "System integration", Sec. 4.5): weights as FDVLM_W_FP8E4M3, and the input rows of the four layer
   * projections (QKV, O, gate/up, down) quantised per token to e4m3 -- scale = max|row| / 448 over the row as stored
   * (f16), code = e4m3(x / scale), float32 quotient, round to nearest even, saturating -- so that those GEMMs run
   * e4m3 x e4m3 on the tensor cores.  The LM head keeps 16-bit input rows.  Needs shapes the tensor-core kernels
   * take (FDVLM_ERR_UNSUPPORTED otherwise).  Of the single operators below only fdvlm_op_linear takes this value. */
  FDVLM_W8A8_FP8E4M3 = 3
} fdvlm_dtype;

/* Element type of the KV cache (and of q, and of the attention probabilities in the P.V product) for the bf16 /
 * fp8 weight types; same bytes either way.  F16 keeps 11 significant bits instead of 8 -- what the stated logit
 * tolerances need at 28-36 layers -- and saturates at +-65504.  Ignored for FDVLM_F32 (fp32 cache). */
typedef enum { FDVLM_KV_BF16 = 0, FDVLM_KV_F16 = 1 } fdvlm_kv_dtype;

typedef struct {
  int n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab;
  int mask_id;        /* id of [MASK]; never predicted (its logit is excluded from softmax/argmax) */
  float rms_eps;      /* RMSNorm epsilon */
  float rope_theta;   /* rotary base; rotate-half pairing (j, j + head_dim/2), position = index in the
                         committed sequence (vision rows included) */
  int tie_embeddings; /* 1: LM head = embedding table (lm_head must be NULL) */
  fdvlm_dtype dtype;
  int max_seq;        /* KV-cache capacity in positions; every call needs cache_len + rows <= max_seq */
  int max_block;      /* largest block size (1..64) */
  fdvlm_kv_dtype kv_dtype;
} fdvlm_config;

typedef struct {
  const void *wq, *wk, *wv, *wo, *w_gate, *w_up, *w_down; /* device, [out,in], storage per dtype */
  const float *bq, *bk, *bv;                              /* device fp32 [out], all NULL or all set */
  const float *s_q, *s_k, *s_v, *s_o, *s_gate, *s_up, *s_down; /* device fp32 [out]; fp8 only    */
  const float *g_attn, *g_mlp;                            /* device fp32 [hidden] RMSNorm gains     */
} fdvlm_layer_weights;

typedef struct {
  const void *embed;      /* device [vocab, hidden], fp32 (F32) or bf16 (BF16 / FP8); never fp8      */
  const void *lm_head;    /* device [vocab, hidden] in dtype storage; NULL iff tie_embeddings        */
  const float *s_lm_head; /* device fp32 [vocab]; fp8 untied only                                   */
  const float *g_final;   /* device fp32 [hidden]                                                   */
  const fdvlm_layer_weights *layers; /* HOST array of n_layers entries (copied by fdvlm_create)     */
} fdvlm_weights;

/* Unmasking rule of one step (Sec. 3.4 / Sec. 4.5).
 *  THRESHOLD: reveal every masked position whose confidence is strictly above `threshold`; if none
 *             is, reveal the single masked position of highest confidence (so tau = 1.0 gives one
 *             token per step).
 *  TOPK:      reveal the min(k, #masked) masked positions of highest confidence.
 *  Ties go to the lowest position index; the vocabulary argmax takes the lowest token id. */
typedef enum { FDVLM_RULE_THRESHOLD = 0, FDVLM_RULE_TOPK = 1 } fdvlm_rule;
/* pred_shift = 0: row i of the forward predicts position i (a block of B masks).  pred_shift = 1: the paper's
 * convention (Appendix B, Alg. 1 "shift-by-one"): row i-1 predicts position i, so position 0 can never be predicted
 * and must be a given token -- the AR seed of Sec. 3.4 "causal context decoding" (pass it through init_tokens). */
typedef struct { fdvlm_rule rule; float threshold; int k; int pred_shift; } fdvlm_step_params;
typedef struct { int n_unmasked, n_remaining, step_index; } fdvlm_step_info;

/* Create a handle on the current CUDA device.  `cuda_stream` is a cudaStream_t (NULL = default
 * stream).  Allocates the KV cache (n_layers * 2 * n_kv_heads * max_seq * head_dim elements) and a
 * workspace.  Requires: head_dim in {64, 128}; n_q_heads % n_kv_heads == 0; hidden, intermediate,
 * q/kv widths multiples of 8 (bf16/fp8: hidden and intermediate multiples of 16); 1 <= max_block <= 64. */
int fdvlm_create(const fdvlm_config *cfg, const fdvlm_weights *w, void *cuda_stream, fdvlm_t **out);
void fdvlm_destroy(fdvlm_t *h);

/* Forget the cache and any open block (cache_len = 0). */
int fdvlm_reset(fdvlm_t *h);

/* Wait for everything issued on the handle's stream and report what the device left in its status word since the
 * last report: FDVLM_ERR_TIMEOUT if a bounded device-side wait gave up, FDVLM_ERR_INVALID_ARG if a token id outside
 * [0, vocab) was met (the embedding of token 0 was used in its place; nothing out of bounds was read), else FDVLM_OK.
 * The asynchronous calls (fdvlm_prefill, fdvlm_commit_block, fdvlm_block_step without `info`) cannot report these
 * themselves; every synchronous call does, and so does this one. */
int fdvlm_synchronize(fdvlm_t *h);

/* Append `n_embeds` embedding rows (device, [n_embeds, hidden], fp32 for F32 else bf16; may be NULL
 * when n_embeds = 0) and then `n_tokens` token ids (device int32; may be NULL when 0) to the cache
 * with a causal forward (Alg. 1 "Prefill (causal attention)").  May be called repeatedly; not inside
 * an open block.  last_logits (device fp32 [vocab], nullable) receives the logits of the last row
 * appended -- the AR seed of Sec. 3.4 "causal context decoding". */
int fdvlm_prefill(fdvlm_t *h, const void *embeds, int n_embeds, const int32_t *tokens, int n_tokens,
                  float *last_logits);

/* Open a block of `block_size` positions at cache_len .. cache_len + block_size - 1.
 * init_tokens (device int32 [block_size], nullable): positions holding mask_id are masked, any other
 * id is an already revealed token; NULL = all masked.  fdvlm_block_begin_host takes a host pointer. */
int fdvlm_block_begin(fdvlm_t *h, int block_size, const int32_t *init_tokens);
int fdvlm_block_begin_host(fdvlm_t *h, int block_size, const int32_t *init_tokens_host);

/* One denoise step over the open block (B = block_size rows).  All outputs nullable:
 *   logits       device fp32 [B, vocab]   raw logits (mask_id column not suppressed)
 *   conf         device fp32 [B]          max softmax probability with mask_id excluded, every row
 *   pred         device int32 [B]         argmax token with mask_id excluded, every row
 *   unmask       device uint8 [B]         1 where a masked position was revealed by this step
 *   block_tokens device int32 [B]         block tokens after the update
 *   info         HOST                     counts after the step; passing it makes the call synchronous
 * Errors: STATE if no block is open or no masked position is left.  The KV cache contents at
 * positions < cache_len are never written by this call. */
int fdvlm_block_step(fdvlm_t *h, const fdvlm_step_params *p, float *logits, float *conf,
                     int32_t *pred, uint8_t *unmask, int32_t *block_tokens, fdvlm_step_info *info);

/* Same step, results copied to HOST buffers (any may be NULL); always synchronous. */
int fdvlm_block_step_host(fdvlm_t *h, const fdvlm_step_params *p, float *conf_host,
                          int32_t *pred_host, uint8_t *unmask_host, int32_t *block_tokens_host,
                          fdvlm_step_info *info);

/* Open a block and run the whole top-k schedule on it without a host round trip between the steps: with k positions
 * revealed per step the number of denoise steps is known in advance (ceil(masked / k)), so all of them are enqueued
 * back to back and the host reads the block state once at the end.  init_tokens as in fdvlm_block_begin (device,
 * nullable); pred_shift as in fdvlm_step_params (with 1, position 0 must be given).  block_tokens (device int32 [B],
 * nullable) receives the finished block; info (HOST, required) the counts after the last step and the number of steps
 * in step_index.  The block is left open and fully revealed: commit it with fdvlm_commit_block(_verify).
 * Errors as fdvlm_block_begin / fdvlm_block_step; STATE if masked positions remain (a masked position 0 under
 * pred_shift = 1). */
int fdvlm_decode_block_topk(fdvlm_t *h, int block_size, const int32_t *init_tokens, int k, int pred_shift,
                            int32_t *block_tokens, fdvlm_step_info *info);

/* Open a block and denoise it to the end under either rule without a host round trip between the steps (Sec. 3.4
 * "confidence-aware parallel decoding": the number of steps of the threshold rule depends on the confidences, so
 * the loop itself runs on the device and stops as soon as no masked position is left).  Arguments as
 * fdvlm_decode_block_topk with the rule in `p`; info (HOST, required) receives the counts after the last step and
 * the number of steps taken in step_index.  Needs a handle created on a non-default stream (the loop is a CUDA graph
 * with a conditional node); UNSUPPORTED otherwise. */
int fdvlm_decode_block(fdvlm_t *h, int block_size, const int32_t *init_tokens, const fdvlm_step_params *p,
                       int32_t *block_tokens, fdvlm_step_info *info);

/* Replace the open block's tokens / masked flags (device int32 [B]; mask_id = masked) without
 * touching the step counter: lets a test replay another implementation's block state. */
int fdvlm_block_set_tokens(fdvlm_t *h, const int32_t *tokens);

/* Commit the open, fully unmasked block: causal forward with cache update, cache_len += B.
 * next_logits (device fp32 [vocab], nullable) = logits of the block's last row.
 * Errors: STATE if no block is open or masked positions remain. */
int fdvlm_commit_block(fdvlm_t *h, float *next_logits);

/* Commit as above and also return, for every row i of the block, the argmax token (mask_id excluded) and its
 * confidence under the causal pass: row_pred[i] is the autoregressive prediction for the position after block row i
 * (Appendix B, Alg. 1 "verify step": a_i = argmax h^v_i).  row_pred device int32 [B], row_conf device fp32 [B],
 * next_logits device fp32 [vocab]; all nullable. */
int fdvlm_commit_block_verify(fdvlm_t *h, int32_t *row_pred, float *row_conf, float *next_logits);

/* fdvlm_commit_block, fdvlm_block_begin and the first fdvlm_block_step of the next block as ONE forward over
 * B_finished + B_next rows (Sec. 3.3: clean context is causal, M_C2C; a noisy block reads the clean context before it,
 * M_N2C, and itself bidirectionally, M_N2N -- the same three masks in one pass): the finished rows run causally among
 * themselves and their K / V land at the positions they are committed to; the next block's rows read the cache, the
 * finished rows and one another.  Results are those of the three calls made one after the other (same arithmetic on
 * other tile shapes); every weight byte is streamed once instead of twice.  Needs B_finished + B_next <=
 * min(max_block, 64) (FDVLM_ERR_CAPACITY otherwise: use the three calls).
 *   next_logits   device fp32 [vocab], nullable: logits of the finished block's last row, as from fdvlm_commit_block
 *   next_init_tokens, p, logits .. info: as for fdvlm_block_begin / fdvlm_block_step, for the next block
 * The _host variant takes and returns host buffers like fdvlm_block_begin_host / fdvlm_block_step_host.
 * Errors: STATE if no block is open or masked positions remain in it; otherwise as the three calls. */
int fdvlm_commit_begin_step(fdvlm_t *h, float *next_logits, int next_block_size, const int32_t *next_init_tokens,
                            const fdvlm_step_params *p, float *logits, float *conf, int32_t *pred, uint8_t *unmask,
                            int32_t *block_tokens, fdvlm_step_info *info);
int fdvlm_commit_begin_step_host(fdvlm_t *h, int next_block_size, const int32_t *next_init_tokens_host,
                                 const fdvlm_step_params *p, float *conf_host, int32_t *pred_host, uint8_t *unmask_host,
                                 int32_t *block_tokens_host, fdvlm_step_info *info);
/* fdvlm_decode_block_topk that first commits the open, fully revealed block, if there is one, in the same forward as the
 * new block's first step (as above); with no block open it is fdvlm_decode_block_topk. */
int fdvlm_commit_decode_block_topk(fdvlm_t *h, int block_size, const int32_t *init_tokens, int k, int pred_shift,
                                   int32_t *block_tokens, fdvlm_step_info *info);
/* The same for fdvlm_decode_block (either rule, loop on the device): the open, fully revealed block is committed in the
 * forward of the new block's first step; the host reads the masked count once after that step (it decides whether the
 * on-device loop runs at all), then once at the end. */
int fdvlm_commit_decode_block(fdvlm_t *h, int block_size, const int32_t *init_tokens, const fdvlm_step_params *p,
                              int32_t *block_tokens, fdvlm_step_info *info);

/* Drop committed positions from the end of the cache: cache_len = new_len (Alg. 1 "Crop").  The dropped K/V rows
 * are simply overwritten by later commits.  Errors: STATE inside an open block; INVALID_ARG unless
 * 0 <= new_len <= cache_len. */
int fdvlm_truncate(fdvlm_t *h, int new_len);

/* One iteration of linear self-speculative decoding (Sec. 3.4 "self-speculative block decoding"; Appendix B,
 * Alg. 1) with block size B: the block [seed, MASK x (B-1)] is drafted in one denoise pass (shift-by-one, every
 * masked position filled), verified by one causal pass with cache update, and the longest prefix on which the
 * causal predictions agree with the draft is accepted: k = 1 + (first j in [0, B-2] with a_j != d_{j+1}; B-1 if
 * none).  The cache keeps block rows 0 .. k-1 (cache_len += k) and a_{k-1} is the next iteration's seed.
 *   seed_token     the block's first token (from fdvlm_prefill's last_logits, or the previous call's next_token)
 *   draft_tokens   device int32 [B], nullable: the block after the draft pass
 *   verify_pred    device int32 [B], nullable: a_0 .. a_{B-1}
 *   info           HOST, required: accepted k, next_token = a_{k-1}, cache_len after the call
 * Always synchronous (the accepted length decides the cache length).  Errors as block_begin / block_step. */
typedef struct { int accepted; int32_t next_token; int cache_len; } fdvlm_spec_info;
int fdvlm_spec_block(fdvlm_t *h, int block_size, int32_t seed_token, int32_t *draft_tokens,
                     int32_t *verify_pred, fdvlm_spec_info *info);

/* ---- quadratic self-speculative decoding (Appendix B, Alg. 2 and the paragraph "Quadratic speculative decoding") ----
 * One forward verifies a draft block d_0 .. d_{B-1} and proposes the next one.  Its input is B groups [d_i, MASK x B];
 * entry j of group i has position id cache_len + i + j; every entry reads the whole cache; (b) the first token of group
 * i reads the first tokens of groups <= i; (c) a mask token of group i reads every entry of group i; (d) nothing else.
 * chain != 0 takes the other reading of (d): a mask token of group i also reads the first tokens of groups < i.
 * P_{i,0} = argmax of group i's first token (the autoregressive prediction for the position after d_i), P_{i,j} = argmax
 * of its j-th mask token (mask_id excluded throughout).  Verify loop: k = 1; while k < B and P_{k-1,0} = d_k: k += 1.
 * d_0 .. d_{k-1} join the sequence, their K / V join the cache (cache_len += k) and P_{k-1,1..B} is the next draft.
 * ROW ORDER of this library (row_pred, logits): rows 0 .. B-1 are the first tokens d_0 .. d_{B-1}, row B + i B + (j-1) is
 * mask token j of group i -- the paper lists the groups one after the other; with the first tokens in front, "keep every
 * (B+1)-th K / V entry" is the first k staging rows of the cache and nothing is moved.
 * The forward has B (B + 1) rows: B (B + 1) <= min(max_block, 64), i.e. B <= 7.
 *
 * fdvlm_quad_begin: Alg. 2 step 1 in cached form.  The prompt is in the cache (fdvlm_prefill); first_token is the token
 *   its last row predicts (argmax of last_logits, mask_id excluded) = d_0; B mask tokens are run in one denoise pass and
 *   the first B-1 of them give d_1 .. d_{B-1} (row i-1 predicts d_i).  The cache is unchanged.  draft: device int32 [B],
 *   nullable.  Synchronous.  Errors: STATE inside an open block; CAPACITY as above or past max_seq; INVALID_ARG.
 * fdvlm_quad_set_draft: overwrite the current draft (device int32 [B]); lets a test replay another implementation's.
 * fdvlm_quad_step: one iteration of the loop.  accepted_tokens device int32 [B] (entries >= accepted are -1), next_draft
 *   device int32 [B], row_pred device int32 [B (B+1)], logits device fp32 [B (B+1), vocab] -- all nullable, in the row
 *   order above; info HOST, required.  Always synchronous (the accepted length decides the cache length).
 * fdvlm_quad_end: leave the mode (the cache keeps what was accepted). */
typedef struct { int accepted; int cache_len; } fdvlm_quad_info;
int fdvlm_quad_begin(fdvlm_t *h, int block_size, int32_t first_token, int chain, int32_t *draft);
int fdvlm_quad_set_draft(fdvlm_t *h, const int32_t *draft);
int fdvlm_quad_step(fdvlm_t *h, int32_t *accepted_tokens, int32_t *next_draft, int32_t *row_pred, float *logits,
                    fdvlm_quad_info *info);
int fdvlm_quad_end(fdvlm_t *h);

/* Committed positions, or a negative status for a NULL handle. */
int fdvlm_cache_len(const fdvlm_t *h);

/* Copy cached K (which = 0, post-rotary) or V (which = 1) of `layer`, positions [pos0, pos0 + n), to
 * dst (device, [n, n_kv_heads, head_dim], fp32 for F32 else the handle's kv_dtype).  For tests and checkpointing. */
int fdvlm_cache_read(const fdvlm_t *h, int layer, int which, int pos0, int n, void *dst);

/* Number of kernel launches issued by the last prefill / step / commit call of this handle. */
int fdvlm_last_launch_count(const fdvlm_t *h);

/* Instrumentation.  mode 0: off.  mode 1: every projection (GEMM) launch group and every attention launch of this
 * handle is bracketed by CUDA events on the handle's stream and the kernels are launched one by one (so without the
 * overlap of the production chain); fdvlm_profile_read synchronises the stream, returns the summed device time
 * (milliseconds) and the number of bracketed groups per family since the last enable / read, and clears the
 * counters.  mode 2 (in-chain timing): the forward runs exactly as in production (graph replay, dependent launches),
 * and every kernel records, from the GPU's global nanosecond timer, the earliest start of any of its CTAs, the
 * earliest return of a CTA from its wait for the predecessor kernel, and the latest end of any CTA;
 * fdvlm_profile_read_chain synchronises and returns the records of the LAST forward in launch order (at most `cap`;
 * *n = how many there were).  Any output pointer may be NULL. */
typedef enum {
  FDVLM_K_ROPE_TABLE = 0, FDVLM_K_GEMM_QKV = 1, FDVLM_K_FIN_QKV = 2, FDVLM_K_ATTENTION = 3, FDVLM_K_ATTN_MERGE = 4,
  FDVLM_K_GEMM_O = 5, FDVLM_K_FIN_RESID = 6, FDVLM_K_GEMM_GATE_UP = 7, FDVLM_K_GEMM_DOWN = 8, FDVLM_K_GEMM_LM_HEAD = 9,
  FDVLM_K_STATS_MERGE = 10
} fdvlm_kernel_kind;
typedef struct { int kind; /* fdvlm_kernel_kind */ double start_us, released_us, end_us; /* relative to the first start */ } fdvlm_kernel_record;
int fdvlm_profile_enable(fdvlm_t *h, int mode);
int fdvlm_profile_read(fdvlm_t *h, double *ms_linear, int *n_linear, double *ms_attention, int *n_attention);
int fdvlm_profile_read_chain(fdvlm_t *h, fdvlm_kernel_record *records, int cap, int *n);

/* Test hook for the give-up path of the kernels' bounded waits.  While `on` is non-zero, every tensor-core GEMM of
 * this handle reads the flag when it starts and each of its roles (TMA producer, MMA issuer, converters, epilogue)
 * leaves at once by the path a timed-out wait takes -- nothing issued, nothing in flight, tensor memory freed -- and
 * records its role in the status word, so the next synchronous call returns FDVLM_ERR_TIMEOUT.  Outputs of such
 * calls are undefined; committed cache positions are not written.  Takes effect in stream order. */
int fdvlm_debug_poison(fdvlm_t *h, int on);

/* Message of the last error on this handle ("" if none); valid until the next call on it.
 * With h = NULL returns the message of the last failed fdvlm_create on this thread. */
const char *fdvlm_last_error(const fdvlm_t *h);

/* ---- a yardstick for measurement (the paper has no counterpart) ---------------------------------------- */

/* Read `bytes` bytes of device memory once, with a plain streaming kernel of this library (16-byte loads, 8 CTAs per SM,
 * nothing written but one 4-byte word at device_sink that the kernel may increment): timed by the caller with CUDA events
 * on a buffer larger than L2, it gives the read-only bandwidth a kernel can reach on this GPU, a second denominator
 * beside the copy bandwidth.  device_buf 16-byte aligned.  Asynchronous on cuda_stream. */
int fdvlm_util_stream_read(const void *device_buf, size_t bytes, void *device_sink, void *cuda_stream);

/* ---- single operators of the path, for kernel-level tests and timing -------------------------------- */

/* y[m, n] = sum_k x[m, k] * w[n, k] (* scale[n]) (+ bias[n]): the small-M weight-streaming GEMM that
 * every projection of the decoder is (QKV, O, gate/up, down, LM head; M = block size <= 64).
 * x: device [m, k], fp32 for F32 else bf16; w: device [n, k] in `dtype` storage; scale: device fp32
 * [n] (fp8) or NULL; bias: device fp32 [n] or NULL; y: device fp32 [m, n].
 * workspace: device scratch of at least fdvlm_op_linear_workspace_bytes(m, n, k, dtype) bytes (never 0): the
 * kernels' status words, split-K partial sums and, for fp8 weights, the f16 copy of x that GEMM multiplies by.
 * The call is asynchronous; fdvlm_op_linear_status(workspace, stream) waits for the stream and returns
 * FDVLM_ERR_TIMEOUT if a bounded wait inside the kernels of the LAST call on that workspace gave up (y is then
 * undefined), else FDVLM_OK.  workspace = NULL asks about the built-in scratch of fdvlm_op_linear_static on the
 * current device.
 * dtype = FDVLM_W8A8_FP8E4M3: w and scale as for fp8 weights; the bf16 rows of x are first stored as f16 (saturating)
 * and each row is then quantised to e4m3 with its own scale max|row| / 448 inside the GEMM kernel, which multiplies
 * e4m3 by e4m3; FDVLM_ERR_UNSUPPORTED where the tensor-core kernel does not take the shape (k not a multiple of 16). */
int fdvlm_op_linear(const void *x, const void *w, const float *scale, const float *bias, float *y,
                    int m, int n, int k, fdvlm_dtype dtype, void *workspace, void *cuda_stream);
size_t fdvlm_op_linear_workspace_bytes(int m, int n, int k, fdvlm_dtype dtype);
int fdvlm_op_linear_status(const void *workspace, void *cuda_stream);

/* (No counterpart in the paper: an integration convenience of this library.)
 * The same projection as fdvlm_op_linear for callers that cannot allocate device memory -- code running
 * under a framework allocator it must not bypass, inside a memory-budgeted plugin, or in a context where
 * cudaMalloc's implicit device synchronisation is not acceptable.  The split-K scratch that
 * fdvlm_op_linear takes as `workspace` is instead a fixed array of FDVLM_STATIC_SCRATCH_BYTES bytes
 * built into the library's device image; every GPU that loads the library holds it until the process
 * exits.  The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   - Shapes whose scratch need (see fdvlm_op_linear_workspace_bytes) exceeds the array are refused with
 *     FDVLM_ERR_CAPACITY; the message (fdvlm_last_error(NULL)) names both sizes.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call before any stream capture.
 *   - All calls on one device share the array: two calls whose kernels may overlap on the GPU (different
 *     streams, no ordering between them) race on it.  Calls on one stream are safe back to back.
 * Arguments, layouts and results are those of fdvlm_op_linear; x, w, scale, bias, y are device pointers
 * owned by the caller.  Errors also set the message returned by fdvlm_last_error(NULL). */
#define FDVLM_STATIC_SCRATCH_BYTES (8u << 20)
int fdvlm_op_linear_static(const void *x, const void *w, const float *scale, const float *bias, float *y,
                           int m, int n, int k, fdvlm_dtype dtype, void *cuda_stream);

/* Block-masked GQA attention of n_rows new rows at positions cache_len .. cache_len + n_rows - 1
 * (Sec. 3.3 masks; Alg. 1 draft / verify).  q: device [n_rows, n_q_heads, head_dim] (post-rotary);
 * k_cache / v_cache: device [n_kv_heads, max_seq, head_dim] holding cache_len committed positions
 * followed by the n_rows new positions; causal = 0: every row reads all cache_len + n_rows keys,
 * causal = 1: row i reads keys 0 .. cache_len + i.  out: device [n_rows, n_q_heads * head_dim].
 * Element type of q, the caches and out: fp32 for F32, otherwise bf16 or f16 as kv_dtype says.  workspace: device
 * scratch of at least fdvlm_op_attention_workspace_bytes(...) bytes for the split-KV partial results. */
int fdvlm_op_attention(const void *q, const void *k_cache, const void *v_cache, void *out,
                       int n_rows, int cache_len, int max_seq, int n_q_heads, int n_kv_heads,
                       int head_dim, int causal, fdvlm_dtype dtype, fdvlm_kv_dtype kv_dtype, void *workspace,
                       void *cuda_stream);
size_t fdvlm_op_attention_workspace_bytes(int n_rows, int n_q_heads, int n_kv_heads, int head_dim);

/* Version string of the library. */
const char *fdvlm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FDVLM_H_ */
