// The request handle behind the C ABI and the helpers shared by its translation units.
#pragma once
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <vector>

#include "../../include/fdvlm.h"
#include "common.cuh"
#include "kernels.h"

struct fdvlm {
  fdvlm_config cfg;
  std::vector<fdvlm_layer_weights> layers;
  fdvlm_weights w;
  cudaStream_t st;
  int device;
  int dt;          // DT_*
  size_t act_sz;   // bytes per activation / KV element
  int act8;        // W8A8: the four layer projections quantise their input rows to e4m3 (weights e4m3 as for DT_FP8)
  int use_tc;      // bf16 / fp8 weights: tcgen05 + TMA GEMMs, tensor-core attention, folded norms
  int kv_type;     // tensor-core path: element type of q and the KV cache (KV_BF16 / KV_F16)
  int xfmt;        // tensor-core path: storage of the GEMM inputs a / ao / act (XF_BF16X2 for bf16 weights, XF_F16 for fp8)
  int head_fmt;    // storage of the LM head's input (as xfmt, but bf16 planes when the head is a tied bf16 table)
  size_t a_lo, ao_lo, act_lo;   // XF_BF16X2: element offset of each buffer's low-order plane
  char* slab;      // one allocation behind every device buffer below except the KV cache
  int32_t* dev_len;   // device copy of cache_len, read by the captured forward graphs
  int use_graphs;     // tensor-core path: replay one captured CUDA graph per (rows, mode, logits mode)
  struct FwdGraph { int n, mode, logits_rows, want_logits, stamped, long_cache, launches; cudaGraphExec_t exec; std::vector<int> kinds; };
  std::vector<FwdGraph> graphs;
  // on-device decode loop (fdvlm_decode_block): a graph whose conditional WHILE node repeats the denoise step
  cudaGraphExec_t loop_exec;
  int loop_n, loop_rule, loop_k, loop_shift, loop_long, loop_body_launches;
  float loop_threshold;
  // device buffers (R = max_block rows)
  char* kv;        // [n_layers][2][Hkv][max_seq][d]
  float* h;        // [R, H] residual stream, fp32
  void* a;         // [R, H] normalised rows (CUDA-core path) / h * gain in bf16 (tensor-core path)
  void* ao;        // [R, Hq*d] attention output
  void* act;       // [R, I]
  void* q;         // [R, Hq*d]
  float* y;        // [R, max((Hq+2Hkv)d, 2I)] fp32 GEMM output (CUDA-core path)
  float* cs;       // [R, d/2] float2 rotary table
  float* ssq;      // [R, nt] partial sums of h^2 per 128 columns (tensor-core path)
  // W8A8: maxima of |value as stored| of the rows of a ([R, nt] partial maxima), ao ([R, Hq] partial maxima) and
  // act ([R], raised atomically by the gate/up epilogue, zeroed by the QKV finalisation of the same layer)
  float* amax_a; float* amax_ao; float* amax_act;
  void* stats;     // [ceil(V/128)*4][R] float4 softmax statistics of the LM-head epilogue
  float* logits;   // [R, V]
  float* conf;     // [R]
  int32_t* pred;   // [R]
  uint8_t* unmask; // [R]
  int32_t* blk_tokens;
  uint8_t* blk_masked;
  int32_t* info;   // {n_unmasked, n_remaining, step_index, device status, poison (host-set test hook),
                   //  iterations of the on-device decode loop, 2 spare}
  int32_t* init_stage;  // [64] device staging of host-given block tokens
  // quadratic self-speculative decoding (Appendix B, Alg. 2): the draft block, and the row masks / position offsets of
  // its B (B + 1)-row forward (MODE_MASKED), written once per fdvlm_quad_begin
  int32_t* q_d;                 // [64] d_0 .. d_{B-1}
  unsigned long long* q_mask;   // [64]
  int* q_pos_off;               // [64]
  int quad_B;                   // 0: no quadratic decode open
  // commit + first step of the next block as one forward (MODE_FUSED): its rows' tokens and row masks
  int32_t* f_rows;              // [64]
  unsigned long long* f_mask;   // [64]
  void* ws;        // GEMM split-K / attention split-KV workspace
  size_t ws_bytes;
  int32_t* info_host;  // pinned
  char* host_stage;    // pinned staging for *_host variants
  int nt;          // ceil(H / 128)
  // state
  int cache_len, block_size, n_remaining, step_index, block_open;
  int launches;
  // optional timing, see fdvlm_profile_*: prof_on = 1: events around each launch group (kernels launched one by one);
  // prof_on = 2: every kernel of the replayed forward stamps the GPU's global timer into `stamps` (in-chain timing)
  int prof_on;
  fdk::KStamp* stamps;                     // device, FDVLM_MAX_STAMPS records
  std::vector<int> stamp_kind;        // kind of each record used by the last stamped forward (fdvlm_kernel_kind)
  int stamp_used;
  std::vector<cudaEvent_t> prof_ev;   // pairs (start, stop)
  std::vector<int> prof_kind;         // per pair: 0 = projection GEMM, 1 = attention
  size_t prof_used;
  char err[512];
};

namespace fdk {

extern thread_local char g_create_error[512];

inline int fail(fdvlm_t* h, int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(h ? h->err : g_create_error, 512, fmt, ap);
  va_end(ap);
  return code;
}
#define CU(h, call)                                                                                 \
  do {                                                                                              \
    cudaError_t e_ = (call);                                                                        \
    if (e_ != cudaSuccess) return fdk::fail(h, FDVLM_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

inline size_t kv_plane(const fdvlm_t* h) {
  return (size_t)h->cfg.n_kv_heads * h->cfg.max_seq * h->cfg.head_dim * h->act_sz;
}
inline char* kv_ptr(const fdvlm_t* h, int layer, int which) { return h->kv + ((size_t)layer * 2 + which) * kv_plane(h); }

inline void prof_begin(fdvlm_t* h, int kind) {
  if (!h->prof_on) return;
  if (h->prof_used * 2 + 2 > h->prof_ev.size()) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { h->prof_on = 0; return; }
    h->prof_ev.push_back(a); h->prof_ev.push_back(b); h->prof_kind.push_back(kind);
  }
  h->prof_kind[h->prof_used] = kind;
  cudaEventRecord(h->prof_ev[h->prof_used * 2], h->st);
}
inline void prof_end(fdvlm_t* h) {
  if (!h->prof_on) return;
  cudaEventRecord(h->prof_ev[h->prof_used * 2 + 1], h->st);
  h->prof_used++;
}

// forward.cu
// Gather n input rows into the residual stream at row `row0`: from the embedding table (tokens, device
// int32) or from caller-given embedding rows (activation type).
int stage_rows(fdvlm_t* h, int row0, int n, const int32_t* tokens, const void* embeds);
// One forward over the n rows staged in the residual stream.  mode: MODE_BIDIR (denoise; Alg. 1 draft
// mask) or MODE_CAUSAL (prefill / commit; Alg. 1 verify mask).  K/V of the rows are staged at cache
// positions cache_len .. cache_len + n - 1; only the caller's increment of cache_len commits them.
// logits_rows: 0 none; n = all rows (logits into h->logits when want_logits, and conf / pred always);
// 1 = last row only, raw logits into h->logits[0 .. V).
int forward_rows(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits);
int forward_rows_enqueue(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits);

size_t linear_workspace_bytes(int m, int n, int k, int dtype);
size_t attention_workspace_bytes(int n, int hq, int hkv, int d);

constexpr int FDVLM_MAX_STAMPS = 1024;
// Bytes at the start of an operator-level workspace that hold the kernels' two status words.
constexpr size_t OP_HEAD = 256;
// Stand-alone projection on `st` (workspace laid out as fdvlm_op_linear documents).  Returns launches or -1.
int launch_linear(const LinearArgs& a, cudaStream_t st, cudaError_t* err);
int launch_attention(const AttnArgs& a, cudaStream_t st, cudaError_t* err);

}  // namespace fdk
