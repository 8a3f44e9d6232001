// Launchers of the fdvlm kernels (host-callable; all asynchronous on `st`).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "common.cuh"

namespace fdk {

// ---- small-M linear: y[m,n] = sum_k x[m,k] w[n,k] (* scale[n]) (+ bias[n]) ---------------------
struct LinearArgs {
  const void* x;        // [m, k]   fp32 (DT_F32) or bf16
  const void* w;        // [n, k]   per dtype
  const float* scale;   // [n] or null
  const float* bias;    // [n] or null
  float* y;             // [m, ldy] fp32 result (written, or accumulated into when `accumulate`)
  int m, n, k, ldy;
  int accumulate;       // 1: y += result (residual add)
  int dtype;            // DT_*
  void* workspace;      // split-K partial sums
  size_t workspace_bytes;
};
size_t linear_workspace_bytes(int m, int n, int k, int dtype);

// ---- elementwise / reduction kernels -----------------------------------------------------------
// tokens outside [0, vocab) read row 0 and leave ST_BAD_TOKEN in *status
void launch_embed(const void* table, const int32_t* tokens, float* h, int n, int hidden, int dtype, int vocab, int* status,
                  cudaStream_t st);
void launch_bf16_to_f16(const void* in, void* out, size_t n, cudaStream_t st);
// the same row by row, leaving amax[row] = max |f16 value| of the row
void launch_bf16_rows_to_f16_amax(const void* in, void* out, int m, int k, float* amax, cudaStream_t st);
void launch_rows_to_f32(const void* rows, float* h, int n, int hidden, int dtype, cudaStream_t st);
void launch_rmsnorm(const float* h, const float* g, void* out, int n, int hidden, float eps, int dtype, cudaStream_t st);
void launch_rope_table(float* cs, int n, int pos0, int head_dim, float theta, cudaStream_t st, const int* len_ptr = nullptr,
                       KStamp* stamp = nullptr, const int* pos_off = nullptr);
// quadratic self-speculative decoding (Appendix B, Alg. 2): row layout, input tokens, first draft, verify loop
// read-only streaming yardstick (see the kernel)
void launch_stream_read(const void* buf, size_t bytes, unsigned* sink, int ctas, cudaStream_t st);
// commit of the finished block + opening of the next one as one forward: rows, row masks, block state
void launch_fuse_begin(int32_t* blk_tokens, uint8_t* blk_masked, int Bc, const int32_t* init, int Bn, int mask_id, int32_t* rows,
                       unsigned long long* mask, int32_t* info, cudaStream_t st);
void launch_quad_layout(int B, int chain, unsigned long long* mask, int* pos_off, cudaStream_t st);
void launch_quad_build(const int32_t* d, int B, int mask_id, int32_t* tokens, uint8_t* masked, cudaStream_t st);
void launch_quad_first_draft(const int32_t* pred, int32_t first, int B, int32_t* d, cudaStream_t st);
void launch_quad_accept(const int32_t* pred, int32_t* d, int B, int32_t* accepted, int32_t* out, cudaStream_t st);
void launch_set_len(int* len_ptr, int value, cudaStream_t st);
// qkv fp32 [n, (Hq + 2 Hkv) d] -> q (act type) [n, Hq, d] rotated; K (rotated) and V written into the
// layer's cache planes [Hkv, max_seq, d] at positions pos0 .. pos0 + n - 1.
void launch_qkv_post(const float* qkv, const float* cs, void* q, void* kc, void* vc, int n, int pos0,
                     int hq, int hkv, int d, int max_seq, int dtype, cudaStream_t st);
void launch_swiglu(const float* gu, void* act, int n, int inter, int dtype, cudaStream_t st);
void launch_row_stats(const float* logits, int n, int vocab, int mask_id, float* conf, int32_t* pred, cudaStream_t st);
// Unmask selection + block-state update.  info = {n_unmasked, n_remaining, step_index}.
// loop = 1: the launch is the last node of a conditional WHILE body; it counts the iteration in info[5] and sets `cond`
// to "masked positions remain".
void launch_select(const float* conf, const int32_t* pred, int32_t* tokens, uint8_t* masked, uint8_t* unmask,
                   int32_t* info, int n, int rule, float threshold, int k, cudaStream_t st, int shift = 0,
                   cudaGraphConditionalHandle cond = 0, int loop = 0);
// out[0] = accepted length k, out[1] = a[k - 1] (Alg. 1 "Accept: left-to-right comparison")
void launch_accept(const int32_t* a, const int32_t* d, int n, int32_t* out, cudaStream_t st);
void launch_init_block(int32_t* tokens, uint8_t* masked, int32_t* info, const int32_t* init, int n, int mask_id,
                       int step, cudaStream_t st);

// ---- tensor-core (tcgen05 + TMA) small-M GEMM, bf16 ---------------------------------------------------
enum { TC_MODE_PARTIAL = 0, TC_MODE_DIRECT = 1, TC_MODE_SWIGLU = 2, TC_MODE_LOGITS = 3 };
// Up to three bf16 matrices that share x and K; their outputs sit side by side in one row of width ld.
struct TcGroup {
  const void* x; int m, k;   // bf16 weights: bf16 rows (hi plane); fp8 weights: f16 rows
  const void* x_lo;          // bf16 weights only, nullable: the rows' low-order bf16 plane (x = hi + lo)
  const void* w[3]; int n[3]; int n_mats;
  const float* scale[3]; const float* bias[3];
  int fp8;   // weights are e4m3 bytes (scale[] holds the per-output-channel factors)
  int a8;    // with fp8: the kernel quantises the f16 rows to e4m3, one scale per row (W8A8); PARTIAL and SWIGLU only
};
// What the GEMM leaves behind.
//   PARTIAL: part[split][m][ld] = split-K partial sums (*splits_out of them) for the caller's reduce kernel
//   DIRECT : y[m][ld] = (x w^T) * rstd[row] * scale + bias (+ y when accumulate)
//   SWIGLU : act[m][n0] = silu(x w0^T * rstd * s0) * (x w1^T * rstd * s1)   (w[0] = gate, w[1] = up)
//   LOGITS : y (when write_logits) as DIRECT, and stats[tile * 4 + quarter][m] = (max, sum exp(l - max), argmax id)
//            over the 32 vocabulary ids a warp holds, mask_id excluded
// rstd[row] = rsqrt(sum_t ssq_in[row][t] / hidden + eps) when ssq_in is set (RMSNorm folded into the consumer), else 1.
struct TcOut {
  int mode;
  float* part; size_t part_bytes; int* splits_out;
  float* y; int ld; int accumulate;
  void* act; size_t act_lo_off; int act_fmt;   // SWIGLU output, stored as XF_* (lo plane act_lo_off elements on)
  const float* ssq_in; int nt_in; int hidden; float eps;
  void* stats; int mask_id; int write_logits;
  int* status;   // two device words: [0] set non-zero if a bounded wait inside the kernel gave up; [1] read at kernel
                 // start, non-zero sends every role down its give-up path at once
  KStamp* stamp; // in-chain timing of the launch, nullable
  // a8 groups: amax_in[row][n_amax_in] = partial maxima of |x[row]| (as stored) left by whoever wrote x; the accumulators
  // are sums of code products, so PARTIAL output still lacks the row's scale max / 448 (the reduce kernel applies it) while
  // SWIGLU applies it itself and raises amax_out[row] (atomic maximum: zero before the launch) to max |act[row]|.
  const float* amax_in; int n_amax_in;
  float* amax_out;
};
// Tensor map of a 2-D row-major [rows, cols] tensor with box {64 columns, box_rows}, zero fill outside the tensor
// (cached per argument set).  kind TM_BF16 / TM_F16: 16-bit elements, 128-byte swizzle; TM_E4M3: bytes, no swizzle;
// TM_E4M3_128: bytes, box of 128 columns, 128-byte swizzle.  False when the driver entry point is missing or the encode fails.
enum { TM_BF16 = 0, TM_E4M3 = 1, TM_F16 = 2, TM_E4M3_128 = 3 };
bool make_tmap(CUtensorMap* tm, const void* ptr, int rows, int cols, int box_rows, int kind = TM_BF16);
bool tc_linear_supported(int m, int n, int k, int dtype);
// Split-K workspace of a group with m rows, output width ld, `tiles` 128-row weight tiles and depth k.
size_t tc_workspace_bytes(int m, int ld, int tiles, int k);
cudaError_t tc_group_launch(const TcGroup& g, const TcOut& o, cudaStream_t st);

// Tensor-core path glue.  ssq[row][nt] holds per-128-column partial sums of h^2; xg / lo_off / fmt: a GEMM input
// stored as XF_* (common.cuh).  q, kc, vc of fin_qkv are KV_BF16 or KV_F16 elements (kv_type).
void launch_embed_prep(const void* table, const int32_t* tokens, const void* rows, float* h, void* xg, size_t lo_off, int fmt,
                       const float* g, float* ssq, int nt, int n, int hidden, int vocab, int* status, cudaStream_t st,
                       KStamp* stamp = nullptr, float* amax = nullptr);
void launch_fin_qkv(const float* part, int S, int m, const float* cs, const float* ssq, int nt, int hidden, float eps,
                    const float* bq, const float* bk, const float* bv, const float* sq, const float* sk, const float* sv, void* q,
                    void* kc, void* vc, int pos0, int hq,
                    int hkv, int d, int max_seq, int kv_type, cudaStream_t st, const int* len_ptr = nullptr, KStamp* stamp = nullptr,
                    const float* amax_in = nullptr, float* amax_zero = nullptr);
void launch_fin_resid(const float* part, int S, int m, int hidden, float* h, const float* g, void* xg, size_t lo_off, int fmt,
                      float* ssq, int nt, const float* scale, cudaStream_t st, KStamp* stamp = nullptr,
                      const float* amax_in = nullptr, int n_amax_in = 0, float* amax_out = nullptr);
void launch_stats_merge(const void* stats, int n_part, int m, float* conf, int32_t* pred, cudaStream_t st, KStamp* stamp = nullptr);

// ---- attention -----------------------------------------------------------------------------------
struct AttnArgs {
  const void* q;   // [n, Hq, d]
  const void* kc;  // [Hkv, max_seq, d]
  const void* vc;
  void* out;       // [n, Hq*d]
  int n, cache_len, max_seq, hq, hkv, d, causal, dtype;
  int kv_type;          // tensor-core kernel: element type of q, kc, vc (KV_BF16 / KV_F16)
  int out_fmt;          // tensor-core kernel: storage of `out` (XF_*), lo plane out_lo_off elements on
  size_t out_lo_off;
  const unsigned long long* row_mask;   // nullable, n <= 64 words: bit r' of word r = row r reads row r' of this forward
                                        // (the cached keys are always read); overrides `causal`
  int long_cache;       // tensor-core kernel: -1 pick the CTA shape from cache_len; 0 / 1 the short- / long-cache shape
                        // (a captured launch serves every later length of its class)
  void* workspace;
  const int* len_ptr;   // nullable: device word holding the cache length (overrides cache_len; tensor-core kernel only)
  int* status;          // nullable: device status words (see TcOut::status)
  float* amax_out;      // nullable (tensor-core kernel): [n][hq] maxima of |out| as stored, per row and head
  KStamp* stamp;        // nullable: two consecutive entries (attention, chunk merge)
};
size_t attention_workspace_bytes(int n, int hq, int hkv, int d);
bool attention_long_cache(int keys);   // whether the tensor-core kernel takes its long-cache shape for this many keys

}  // namespace fdk
