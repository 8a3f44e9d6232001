// Host side of the C ABI: handle, state machine, argument checks, and the per-forward launch
// sequence (Fast-dVLM Sec. 3.4 decode loop; Appendix B Alg. 1 for the two forward modes).
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/fdvlm.h"
#include "common.cuh"
#include "kernels.h"

using namespace fdk;

namespace fdk {
int launch_linear_simt(const LinearArgs& a, cudaStream_t st, cudaError_t* err);
size_t simt_workspace_bytes(int m, int n, int k);
int launch_attention_simt(const AttnArgs& a, cudaStream_t st, cudaError_t* err);

void launch_splitk_epilogue(const float* part, int S, int m, int n, const float* scale, const float* bias, float* y, int ldy,
                            int accumulate, cudaStream_t st);

// Device word shared by the stand-alone operator entry points for the kernels' timeout reports.
static int* op_status_word() {
  static int* w = nullptr;
  if (!w) {
    if (cudaMalloc((void**)&w, sizeof(int)) != cudaSuccess) return nullptr;
    cudaMemset(w, 0, sizeof(int));
  }
  return w;
}

size_t linear_workspace_bytes(int m, int n, int k, int dtype) {
  size_t a = simt_workspace_bytes(m, n, k);
  size_t b = tc_linear_supported(m, n, k, dtype) ? tc_workspace_bytes(m, n, (n + 127) / 128, k) : 0;
  return a > b ? a : b;
}
// One projection y = x w^T (* scale) (+ bias) (+ y): bf16 weights go to the tensor-core kernel
// (split-K partial sums + fixed-order reduction), everything else to the CUDA-core kernel.
int launch_linear(const LinearArgs& a, cudaStream_t st, cudaError_t* err) {
  if (!tc_linear_supported(a.m, a.n, a.k, a.dtype)) return launch_linear_simt(a, st, err);
  TcGroup g;
  memset(&g, 0, sizeof(g));
  g.x = a.x; g.m = a.m; g.k = a.k; g.w[0] = a.w; g.n[0] = a.n; g.n_mats = 1;
  int splits = 0;
  int* status = op_status_word();
  if (!status || !a.workspace) { *err = cudaErrorInvalidValue; return -1; }
  *err = tc_group_launch(g, TC_MODE_PARTIAL, (float*)a.workspace, a.workspace_bytes, &splits, nullptr, a.n, 0, nullptr, status, st);
  if (*err != cudaSuccess) return -1;
  launch_splitk_epilogue((const float*)a.workspace, splits, a.m, a.n, a.scale, a.bias, a.y, a.ldy, a.accumulate, st);
  *err = cudaGetLastError();
  return *err == cudaSuccess ? 2 : -1;
}
size_t attention_mma_workspace_bytes(int n, int hq, int hkv, int d);
int launch_attention_mma(const AttnArgs& a, cudaStream_t st, cudaError_t* err);
size_t attention_workspace_bytes(int n, int hq, int hkv, int d) { return attention_mma_workspace_bytes(n, hq, hkv, d); }
// bf16 rows go to the split-KV tensor-core kernel, fp32 rows to the exact CUDA-core kernel.
int launch_attention(const AttnArgs& a, cudaStream_t st, cudaError_t* err) {
  return a.dtype == DT_F32 ? launch_attention_simt(a, st, err) : launch_attention_mma(a, st, err);
}
}  // namespace fdk

static thread_local char g_create_error[512] = "";

struct fdvlm {
  fdvlm_config cfg;
  std::vector<fdvlm_layer_weights> layers;
  fdvlm_weights w;
  cudaStream_t st;
  int device;
  int dt;          // DT_*
  size_t act_sz;   // bytes per activation / KV element
  // fused per-layer weights are not repacked: q, k, v are three GEMMs into one [R, (Hq+2Hkv)d] buffer
  // device buffers
  char* kv;        // [n_layers][2][Hkv][max_seq][d]
  float* h;        // [R, H] residual stream, fp32
  void* a;         // [R, max(H, Hq*d)] normalised rows / attention output
  void* act;       // [R, I]
  void* q;         // [R, Hq*d]
  float* y;        // [R, max((Hq+2Hkv)d, 2I)] fp32 GEMM output
  float* cs;       // [R, d/2] float2 rotary table
  float* logits;   // [R, V]
  float* conf;     // [R]
  int32_t* pred;   // [R]
  uint8_t* unmask; // [R]
  int32_t* blk_tokens;
  uint8_t* blk_masked;
  int32_t* info;   // 4 ints
  int32_t* init_stage;  // [64] device staging of host-given block tokens
  void* ws;        // GEMM / attention workspace
  size_t ws_bytes;
  int32_t* info_host;  // pinned
  char* host_stage;    // pinned staging for *_host variants
  // state
  int cache_len, block_size, n_remaining, step_index, block_open;
  int launches;
  int use_tc;      // bf16 weights on the tcgen05 + TMA kernels
  // optional per-kernel-family timing (events around each launch group), see fdvlm_profile_*
  int prof_on;
  std::vector<cudaEvent_t> prof_ev;   // pairs (start, stop)
  std::vector<int> prof_kind;         // per pair: 0 = linear, 1 = attention
  size_t prof_used;
  char err[512];
};

static void prof_begin(fdvlm_t* h, int kind) {
  if (!h->prof_on) return;
  if (h->prof_used * 2 + 2 > h->prof_ev.size()) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { h->prof_on = 0; return; }
    h->prof_ev.push_back(a); h->prof_ev.push_back(b); h->prof_kind.push_back(kind);
  }
  h->prof_kind[h->prof_used] = kind;
  cudaEventRecord(h->prof_ev[h->prof_used * 2], h->st);
}
static void prof_end(fdvlm_t* h) {
  if (!h->prof_on) return;
  cudaEventRecord(h->prof_ev[h->prof_used * 2 + 1], h->st);
  h->prof_used++;
}

static int fail(fdvlm_t* h, int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(h ? h->err : g_create_error, 512, fmt, ap);
  va_end(ap);
  return code;
}
#define CU(h, call)                                                                              \
  do {                                                                                           \
    cudaError_t e_ = (call);                                                                     \
    if (e_ != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

static size_t kv_plane(const fdvlm_t* h) { return (size_t)h->cfg.n_kv_heads * h->cfg.max_seq * h->cfg.head_dim * h->act_sz; }
static char* kv_ptr(const fdvlm_t* h, int layer, int which) { return h->kv + ((size_t)layer * 2 + which) * kv_plane(h); }

static int check_config(const fdvlm_config* c) {
  if (c->n_layers < 1 || c->hidden < 8 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->intermediate < 8 || c->vocab < 2)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "config: non-positive dimension");
  if (c->head_dim != 64 && c->head_dim != 128) return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (c->n_q_heads % c->n_kv_heads) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "n_q_heads not a multiple of n_kv_heads");
  if (c->dtype != FDVLM_F32 && c->dtype != FDVLM_BF16 && c->dtype != FDVLM_W_FP8E4M3)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "unknown dtype %d", (int)c->dtype);
  int mult = c->dtype == FDVLM_F32 ? 8 : 16;
  if (c->hidden % mult || c->intermediate % mult)
    return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "hidden and intermediate must be multiples of %d", mult);
  if (c->mask_id < 0 || c->mask_id >= c->vocab) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "mask_id out of range");
  if (c->max_block < 1 || c->max_block > 64) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "max_block must be in 1..64");
  if (c->max_seq < c->max_block) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "max_seq smaller than max_block");
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 0.f)) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "rms_eps / rope_theta must be positive");
  return FDVLM_OK;
}

extern "C" const char* fdvlm_version(void) { return "fdvlm 0.1 (sm_100a)"; }

extern "C" const char* fdvlm_last_error(const fdvlm_t* h) { return h ? h->err : g_create_error; }

extern "C" void fdvlm_destroy(fdvlm_t* h) {
  if (!h) return;
  void* bufs[] = {h->kv, h->h, h->a, h->act, h->q, h->y, h->cs, h->logits, h->conf, h->pred, h->unmask,
                  h->blk_tokens, h->blk_masked, h->info, h->init_stage, h->ws};
  for (void* p : bufs) if (p) cudaFree(p);
  for (cudaEvent_t ev : h->prof_ev) cudaEventDestroy(ev);
  if (h->info_host) cudaFreeHost(h->info_host);
  if (h->host_stage) cudaFreeHost(h->host_stage);
  delete h;
}

extern "C" int fdvlm_create(const fdvlm_config* cfg, const fdvlm_weights* w, void* cuda_stream, fdvlm_t** out) {
  g_create_error[0] = 0;
  if (!cfg || !w || !out) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "NULL argument");
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!w->embed || !w->g_final || !w->layers) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "weights: NULL embed / g_final / layers");
  if (cfg->tie_embeddings ? (w->lm_head != nullptr) : (w->lm_head == nullptr))
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "lm_head must be NULL exactly when tie_embeddings is set");
  if (cfg->dtype == FDVLM_W_FP8E4M3 && !cfg->tie_embeddings && !w->s_lm_head)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "fp8 lm_head needs s_lm_head");
  for (int l = 0; l < cfg->n_layers; ++l) {
    const fdvlm_layer_weights& lw = w->layers[l];
    if (!lw.wq || !lw.wk || !lw.wv || !lw.wo || !lw.w_gate || !lw.w_up || !lw.w_down || !lw.g_attn || !lw.g_mlp)
      return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: NULL weight", l);
    int nb = (lw.bq != nullptr) + (lw.bk != nullptr) + (lw.bv != nullptr);
    if (nb != 0 && nb != 3) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: biases must be all NULL or all set", l);
    if (cfg->dtype == FDVLM_W_FP8E4M3 && (!lw.s_q || !lw.s_k || !lw.s_v || !lw.s_o || !lw.s_gate || !lw.s_up || !lw.s_down))
      return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: fp8 weights need all scales", l);
  }
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev == 0) return fail(nullptr, FDVLM_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(e));

  fdvlm_t* h = new (std::nothrow) fdvlm;
  if (!h) return fail(nullptr, FDVLM_ERR_OOM, "host allocation failed");
  memset(&h->cfg, 0, sizeof(h->cfg));
  h->cfg = *cfg;
  h->layers.assign(w->layers, w->layers + cfg->n_layers);
  h->w = *w;
  h->w.layers = h->layers.data();
  h->st = (cudaStream_t)cuda_stream;
  h->dt = (int)cfg->dtype;
  h->act_sz = cfg->dtype == FDVLM_F32 ? 4 : 2;
  h->err[0] = 0;
  h->cache_len = h->block_size = h->n_remaining = h->step_index = h->block_open = 0;
  h->launches = 0;
  h->prof_on = 0;
  h->prof_used = 0;
  h->kv = nullptr; h->h = nullptr; h->a = h->act = h->q = nullptr; h->y = nullptr; h->cs = nullptr; h->logits = nullptr;
  h->conf = nullptr; h->pred = nullptr; h->unmask = nullptr; h->blk_tokens = nullptr; h->blk_masked = nullptr;
  h->info = nullptr; h->init_stage = nullptr; h->ws = nullptr; h->info_host = nullptr; h->host_stage = nullptr;
  cudaGetDevice(&h->device);

  const int R = cfg->max_block, H = cfg->hidden, I = cfg->intermediate, d = cfg->head_dim;
  const int NQ = cfg->n_q_heads * d, NKV = cfg->n_kv_heads * d, NQKV = NQ + 2 * NKV;
  size_t ws = 0;
  const int shapes[][2] = {{NQ, H}, {NKV, H}, {H, NQ}, {I, H}, {H, I}, {cfg->vocab, H}};
  for (auto& s : shapes) { size_t b = linear_workspace_bytes(R, s[0], s[1], h->dt); if (b > ws) ws = b; }
  size_t wa = attention_workspace_bytes(R, cfg->n_q_heads, cfg->n_kv_heads, d);
  if (wa > ws) ws = wa;
  h->use_tc = (h->dt == DT_BF16) && tc_linear_supported(R, NQ, H, DT_BF16);
  if (h->use_tc) {
    const size_t g3[] = {tc_workspace_bytes(R, NQKV, (NQ + 127) / 128 + 2 * ((NKV + 127) / 128), H),
                         tc_workspace_bytes(R, H, (H + 127) / 128, NQ), tc_workspace_bytes(R, H, (H + 127) / 128, I)};
    for (size_t b : g3) if (b > ws) ws = b;
  }
  h->ws_bytes = ws;
  struct { void** p; size_t bytes; } allocs[] = {
      {(void**)&h->kv, (size_t)cfg->n_layers * 2 * kv_plane(h)},
      {(void**)&h->h, (size_t)R * H * 4},
      {(void**)&h->a, (size_t)R * (H > NQ ? H : NQ) * h->act_sz},
      {(void**)&h->act, (size_t)R * I * h->act_sz},
      {(void**)&h->q, (size_t)R * NQ * h->act_sz},
      {(void**)&h->y, (size_t)R * (NQKV > 2 * I ? NQKV : 2 * I) * 4},
      {(void**)&h->cs, (size_t)R * d * 4},
      {(void**)&h->logits, (size_t)R * cfg->vocab * 4},
      {(void**)&h->conf, (size_t)R * 4},
      {(void**)&h->pred, (size_t)R * 4},
      {(void**)&h->unmask, 64},
      {(void**)&h->blk_tokens, 64 * 4},
      {(void**)&h->blk_masked, 64},
      {(void**)&h->info, 16},
      {(void**)&h->init_stage, 64 * 4},
      {(void**)&h->ws, ws ? ws : 16},
  };
  for (auto& a : allocs) {
    e = cudaMalloc(a.p, a.bytes);
    if (e != cudaSuccess) {
      fail(nullptr, FDVLM_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", a.bytes, cudaGetErrorString(e));
      cudaGetLastError();
      fdvlm_destroy(h);
      return FDVLM_ERR_OOM;
    }
  }
  if (cudaMallocHost((void**)&h->info_host, 16) != cudaSuccess || cudaMallocHost((void**)&h->host_stage, 64 * 16) != cudaSuccess) {
    fail(nullptr, FDVLM_ERR_OOM, "pinned host allocation failed");
    fdvlm_destroy(h);
    return FDVLM_ERR_OOM;
  }
  e = cudaMemsetAsync(h->kv, 0, (size_t)cfg->n_layers * 2 * kv_plane(h), h->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->info, 0, 16, h->st);
  if (e != cudaSuccess) {
    fail(nullptr, FDVLM_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    fdvlm_destroy(h);
    return FDVLM_ERR_CUDA;
  }
  *out = h;
  return FDVLM_OK;
}

extern "C" int fdvlm_reset(fdvlm_t* h) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  h->cache_len = 0;
  h->block_open = 0;
  h->block_size = h->n_remaining = h->step_index = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_cache_len(const fdvlm_t* h) { return h ? h->cache_len : (int)FDVLM_ERR_INVALID_ARG; }
extern "C" int fdvlm_last_launch_count(const fdvlm_t* h) { return h ? h->launches : (int)FDVLM_ERR_INVALID_ARG; }

static int forward_rows_tc(fdvlm_t* h, int n, int mode, int logits_rows);

// ---- one forward over n rows already gathered into h->h -------------------------------------------
// mode: MODE_BIDIR (denoise; Alg. 1 draft mask) or MODE_CAUSAL (prefill / commit; Alg. 1 verify mask).
// K/V of the n rows are always staged at cache positions cache_len .. cache_len + n - 1; only the
// caller's later increment of cache_len makes them part of the committed cache.
// logits_rows: 0 = none, n = all rows into h->logits, 1 = last row only into h->logits[0..V).
static int forward_rows(fdvlm_t* h, int n, int mode, int logits_rows) {
  const fdvlm_config& c = h->cfg;
  const int H = c.hidden, I = c.intermediate, d = c.head_dim;
  const int NQ = c.n_q_heads * d, NKV = c.n_kv_heads * d, NQKV = NQ + 2 * NKV;
  cudaError_t e = cudaSuccess;
  if (h->use_tc) return forward_rows_tc(h, n, mode, logits_rows);
  auto lin = [&](const void* x, const void* w, const float* scale, const float* bias, float* y, int nn, int kk, int ldy,
                 int accumulate, int m) -> int {
    LinearArgs a;
    a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = nn; a.k = kk; a.ldy = ldy;
    a.accumulate = accumulate; a.dtype = h->dt; a.workspace = h->ws; a.workspace_bytes = h->ws_bytes;
    prof_begin(h, 0);
    int r = launch_linear(a, h->st, &e);
    prof_end(h);
    if (r < 0) return -1;
    h->launches += r;
    return 0;
  };
  launch_rope_table(h->cs, n, h->cache_len, d, c.rope_theta, h->st);
  h->launches++;
  for (int l = 0; l < c.n_layers; ++l) {
    const fdvlm_layer_weights& lw = h->layers[l];
    launch_rmsnorm(h->h, lw.g_attn, h->a, n, H, c.rms_eps, h->dt, h->st);
    if (lin(h->a, lw.wq, lw.s_q, lw.bq, h->y, NQ, H, NQKV, 0, n) || lin(h->a, lw.wk, lw.s_k, lw.bk, h->y + NQ, NKV, H, NQKV, 0, n) ||
        lin(h->a, lw.wv, lw.s_v, lw.bv, h->y + NQ + NKV, NKV, H, NQKV, 0, n))
      return fail(h, FDVLM_ERR_CUDA, "qkv projection launch: %s", cudaGetErrorString(e));
    launch_qkv_post(h->y, h->cs, h->q, kv_ptr(h, l, 0), kv_ptr(h, l, 1), n, h->cache_len, c.n_q_heads, c.n_kv_heads, d,
                    c.max_seq, h->dt, h->st);
    AttnArgs at;
    at.q = h->q; at.kc = kv_ptr(h, l, 0); at.vc = kv_ptr(h, l, 1); at.out = h->a; at.n = n; at.cache_len = h->cache_len;
    at.max_seq = c.max_seq; at.hq = c.n_q_heads; at.hkv = c.n_kv_heads; at.d = d; at.causal = (mode == MODE_CAUSAL);
    at.dtype = h->dt; at.workspace = h->ws;
    prof_begin(h, 1);
    int r = launch_attention(at, h->st, &e);
    prof_end(h);
    if (r < 0) return fail(h, FDVLM_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    h->launches += r + 2;
    if (lin(h->a, lw.wo, lw.s_o, nullptr, h->h, H, NQ, H, 1, n))
      return fail(h, FDVLM_ERR_CUDA, "o projection launch: %s", cudaGetErrorString(e));
    launch_rmsnorm(h->h, lw.g_mlp, h->a, n, H, c.rms_eps, h->dt, h->st);
    if (lin(h->a, lw.w_gate, lw.s_gate, nullptr, h->y, I, H, 2 * I, 0, n) || lin(h->a, lw.w_up, lw.s_up, nullptr, h->y + I, I, H, 2 * I, 0, n))
      return fail(h, FDVLM_ERR_CUDA, "gate/up projection launch: %s", cudaGetErrorString(e));
    launch_swiglu(h->y, h->act, n, I, h->dt, h->st);
    if (lin(h->act, lw.w_down, lw.s_down, nullptr, h->h, H, I, H, 1, n))
      return fail(h, FDVLM_ERR_CUDA, "down projection launch: %s", cudaGetErrorString(e));
    h->launches += 2;
  }
  if (logits_rows > 0) {
    const int first = (logits_rows == n) ? 0 : n - 1;
    const int m = n - first;
    launch_rmsnorm(h->h + (size_t)first * H, h->w.g_final, h->a, m, H, c.rms_eps, h->dt, h->st);
    h->launches++;
    const void* table = c.tie_embeddings ? h->w.embed : h->w.lm_head;
    const float* sc = c.tie_embeddings ? nullptr : h->w.s_lm_head;
    // a tied table is stored in the embedding's type: fp32 for F32, bf16 otherwise (never fp8)
    int saved = h->dt;
    if (c.tie_embeddings && h->dt == DT_FP8) h->dt = DT_BF16;
    int rc = lin(h->a, table, sc, nullptr, h->logits, c.vocab, H, c.vocab, 0, m);
    h->dt = saved;
    if (rc) return fail(h, FDVLM_ERR_CUDA, "lm head launch: %s", cudaGetErrorString(e));
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

// The same forward on the tensor-core path (bf16 weights): per layer
//   [QKV GEMM -> split-K partials] [reduce + bias + rotary + K/V staging] [attention]
//   [O GEMM -> partials] [reduce + residual + RMSNorm] [gate/up GEMM with SwiGLU epilogue]
//   [down GEMM -> partials] [reduce + residual + next RMSNorm]
// and the LM head as one GEMM writing fp32 logits.
static int forward_rows_tc(fdvlm_t* h, int n, int mode, int logits_rows) {
  const fdvlm_config& c = h->cfg;
  const int H = c.hidden, I = c.intermediate, d = c.head_dim;
  const int NQ = c.n_q_heads * d, NKV = c.n_kv_heads * d, NQKV = NQ + 2 * NKV;
  int* status = h->info + 3;
  float* part = (float*)h->ws;
  cudaError_t e = cudaSuccess;
  auto group = [&](const void* x, int k, int nm, const void* w0, int n0, const void* w1, int n1, const void* w2, int n2) {
    TcGroup g;
    memset(&g, 0, sizeof(g));
    g.x = x; g.m = n; g.k = k; g.n_mats = nm;
    g.w[0] = w0; g.n[0] = n0; g.w[1] = w1; g.n[1] = n1; g.w[2] = w2; g.n[2] = n2;
    return g;
  };
  launch_rope_table(h->cs, n, h->cache_len, d, c.rope_theta, h->st);
  launch_reduce_residual_rmsnorm(nullptr, 0, n, H, nullptr, h->h, h->layers[0].g_attn, h->a, c.rms_eps, h->st);
  h->launches += 2;
  for (int l = 0; l < c.n_layers; ++l) {
    const fdvlm_layer_weights& lw = h->layers[l];
    int S = 0;
    TcGroup g = group(h->a, H, 3, lw.wq, NQ, lw.wk, NKV, lw.wv, NKV);
    prof_begin(h, 0);
    e = tc_group_launch(g, TC_MODE_PARTIAL, part, h->ws_bytes, &S, nullptr, NQKV, 0, nullptr, status, h->st);
    prof_end(h);
    if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "qkv projection launch: %s", cudaGetErrorString(e));
    launch_qkv_reduce_rope(part, S, n, h->cs, nullptr, nullptr, nullptr, lw.bq, lw.bk, lw.bv, h->q, kv_ptr(h, l, 0),
                           kv_ptr(h, l, 1), h->cache_len, c.n_q_heads, c.n_kv_heads, d, c.max_seq, h->st);
    AttnArgs at;
    at.q = h->q; at.kc = kv_ptr(h, l, 0); at.vc = kv_ptr(h, l, 1); at.out = h->a; at.n = n; at.cache_len = h->cache_len;
    at.max_seq = c.max_seq; at.hq = c.n_q_heads; at.hkv = c.n_kv_heads; at.d = d; at.causal = (mode == MODE_CAUSAL);
    at.dtype = h->dt; at.workspace = h->ws;
    prof_begin(h, 1);
    int r = launch_attention(at, h->st, &e);
    prof_end(h);
    if (r < 0) return fail(h, FDVLM_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    h->launches += r + 2;
    g = group(h->a, NQ, 1, lw.wo, H, nullptr, 0, nullptr, 0);
    prof_begin(h, 0);
    e = tc_group_launch(g, TC_MODE_PARTIAL, part, h->ws_bytes, &S, nullptr, H, 0, nullptr, status, h->st);
    prof_end(h);
    if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "o projection launch: %s", cudaGetErrorString(e));
    launch_reduce_residual_rmsnorm(part, S, n, H, nullptr, h->h, lw.g_mlp, h->a, c.rms_eps, h->st);
    g = group(h->a, H, 2, lw.w_gate, I, lw.w_up, I, nullptr, 0);
    prof_begin(h, 0);
    e = tc_group_launch(g, TC_MODE_SWIGLU, nullptr, 0, nullptr, nullptr, 0, 0, h->act, status, h->st);
    prof_end(h);
    if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "gate/up projection launch: %s", cudaGetErrorString(e));
    g = group(h->act, I, 1, lw.w_down, H, nullptr, 0, nullptr, 0);
    prof_begin(h, 0);
    e = tc_group_launch(g, TC_MODE_PARTIAL, part, h->ws_bytes, &S, nullptr, H, 0, nullptr, status, h->st);
    prof_end(h);
    if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "down projection launch: %s", cudaGetErrorString(e));
    const float* g_next = (l + 1 < c.n_layers) ? h->layers[l + 1].g_attn : h->w.g_final;
    launch_reduce_residual_rmsnorm(part, S, n, H, nullptr, h->h, g_next, h->a, c.rms_eps, h->st);
    h->launches += 5;
  }
  if (logits_rows > 0) {
    const int first = (logits_rows == n) ? 0 : n - 1;
    const void* table = c.tie_embeddings ? h->w.embed : h->w.lm_head;
    TcGroup g = group((const char*)h->a + (size_t)first * H * 2, H, 1, table, c.vocab, nullptr, 0, nullptr, 0);
    g.m = n - first;
    prof_begin(h, 0);
    e = tc_group_launch(g, TC_MODE_DIRECT, nullptr, 0, nullptr, h->logits, c.vocab, 0, nullptr, status, h->st);
    prof_end(h);
    if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "lm head launch: %s", cudaGetErrorString(e));
    h->launches++;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

extern "C" int fdvlm_prefill(fdvlm_t* h, const void* embeds, int n_embeds, const int32_t* tokens, int n_tokens,
                             float* last_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (n_embeds < 0 || n_tokens < 0 || (n_embeds > 0 && !embeds) || (n_tokens > 0 && !tokens))
    return fail(h, FDVLM_ERR_INVALID_ARG, "prefill: negative count or NULL rows");
  if (h->block_open) return fail(h, FDVLM_ERR_STATE, "prefill inside an open block");
  const int total = n_embeds + n_tokens;
  if (total == 0) return last_logits ? fail(h, FDVLM_ERR_INVALID_ARG, "prefill: no rows but logits requested") : FDVLM_OK;
  if ((long long)h->cache_len + total > h->cfg.max_seq)
    return fail(h, FDVLM_ERR_CAPACITY, "prefill: %d + %d rows exceed max_seq %d", h->cache_len, total, h->cfg.max_seq);
  h->launches = 0;
  const int R = h->cfg.max_block, H = h->cfg.hidden;
  int done = 0;
  while (done < total) {
    int n = total - done < R ? total - done : R;
    // rows [done, done+n): embeddings first, then tokens
    int ne = 0;
    if (done < n_embeds) {
      ne = n_embeds - done < n ? n_embeds - done : n;
      launch_rows_to_f32((const char*)embeds + (size_t)done * H * h->act_sz, h->h, ne, H, h->dt == DT_F32 ? DT_F32 : DT_BF16, h->st);
      h->launches++;
    }
    if (ne < n) {
      int t0 = done + ne - n_embeds;
      launch_embed(h->w.embed, tokens + t0, h->h + (size_t)ne * H, n - ne, H, h->dt == DT_F32 ? DT_F32 : DT_BF16, h->st);
      h->launches++;
    }
    bool last = (done + n == total);
    int rc = forward_rows(h, n, MODE_CAUSAL, (last && last_logits) ? 1 : 0);
    if (rc) return rc;
    h->cache_len += n;
    done += n;
  }
  if (last_logits) CU(h, cudaMemcpyAsync(last_logits, h->logits, (size_t)h->cfg.vocab * 4, cudaMemcpyDeviceToDevice, h->st));
  return FDVLM_OK;
}

static int block_begin_common(fdvlm_t* h, int block_size) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (block_size < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "block_size must be positive");
  if (block_size > h->cfg.max_block) return fail(h, FDVLM_ERR_CAPACITY, "block_size %d exceeds max_block %d", block_size, h->cfg.max_block);
  if (h->block_open) return fail(h, FDVLM_ERR_STATE, "a block is already open");
  if (h->cache_len + block_size > h->cfg.max_seq)
    return fail(h, FDVLM_ERR_CAPACITY, "block: %d + %d exceed max_seq %d", h->cache_len, block_size, h->cfg.max_seq);
  return FDVLM_OK;
}

static int sync_info(fdvlm_t* h) {
  CU(h, cudaMemcpyAsync(h->info_host, h->info, 16, cudaMemcpyDeviceToHost, h->st));
  CU(h, cudaStreamSynchronize(h->st));
  h->n_remaining = h->info_host[1];
  if (h->info_host[3] != 0) {
    int code = h->info_host[3];
    cudaMemsetAsync(h->info + 3, 0, 4, h->st);
    return fail(h, FDVLM_ERR_TIMEOUT, "a bounded device-side wait gave up (kernel role %d); results of this call are invalid", code);
  }
  return FDVLM_OK;
}

extern "C" int fdvlm_block_begin(fdvlm_t* h, int block_size, const int32_t* init_tokens) {
  int rc = block_begin_common(h, block_size);
  if (rc) return rc;
  launch_init_block(h->blk_tokens, h->blk_masked, h->info, init_tokens, block_size, h->cfg.mask_id, 0, h->st);
  CU(h, cudaGetLastError());
  h->block_open = 1;
  h->block_size = block_size;
  h->step_index = 0;
  if (init_tokens) return sync_info(h);
  h->n_remaining = block_size;
  return FDVLM_OK;
}

extern "C" int fdvlm_block_begin_host(fdvlm_t* h, int block_size, const int32_t* init_tokens_host) {
  int rc = block_begin_common(h, block_size);
  if (rc) return rc;
  if (!init_tokens_host) return fdvlm_block_begin(h, block_size, nullptr);
  memcpy(h->host_stage, init_tokens_host, (size_t)block_size * 4);
  CU(h, cudaMemcpyAsync(h->init_stage, h->host_stage, (size_t)block_size * 4, cudaMemcpyHostToDevice, h->st));
  return fdvlm_block_begin(h, block_size, h->init_stage);
}

extern "C" int fdvlm_block_set_tokens(fdvlm_t* h, const int32_t* tokens) {
  if (!h || !tokens) return h ? fail(h, FDVLM_ERR_INVALID_ARG, "NULL tokens") : (int)FDVLM_ERR_INVALID_ARG;
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "no open block");
  launch_init_block(h->blk_tokens, h->blk_masked, h->info, tokens, h->block_size, h->cfg.mask_id, h->step_index, h->st);
  CU(h, cudaGetLastError());
  return sync_info(h);
}

static int step_core(fdvlm_t* h, const fdvlm_step_params* p) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!p) return fail(h, FDVLM_ERR_INVALID_ARG, "NULL step params");
  if (p->rule != FDVLM_RULE_THRESHOLD && p->rule != FDVLM_RULE_TOPK) return fail(h, FDVLM_ERR_INVALID_ARG, "unknown rule");
  if (p->rule == FDVLM_RULE_TOPK && p->k < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "top-k needs k >= 1");
  if (p->rule == FDVLM_RULE_THRESHOLD && !(p->threshold == p->threshold)) return fail(h, FDVLM_ERR_INVALID_ARG, "threshold is NaN");
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "block_step without an open block");
  if (h->n_remaining == 0) return fail(h, FDVLM_ERR_STATE, "block_step with no masked position left");
  const int B = h->block_size;
  h->launches = 0;
  launch_embed(h->w.embed, h->blk_tokens, h->h, B, h->cfg.hidden, h->dt == DT_F32 ? DT_F32 : DT_BF16, h->st);
  h->launches++;
  int rc = forward_rows(h, B, MODE_BIDIR, B);
  if (rc) return rc;
  launch_row_stats(h->logits, B, h->cfg.vocab, h->cfg.mask_id, h->conf, h->pred, h->st);
  launch_select(h->conf, h->pred, h->blk_tokens, h->blk_masked, h->unmask, h->info, B, (int)p->rule, p->threshold, p->k, h->st);
  h->launches += 2;
  CU(h, cudaGetLastError());
  h->step_index++;
  return FDVLM_OK;
}

static int finish_info(fdvlm_t* h, fdvlm_step_info* info) {
  int rc = sync_info(h);
  if (rc) return rc;
  if (info) { info->n_unmasked = h->info_host[0]; info->n_remaining = h->info_host[1]; info->step_index = h->info_host[2]; }
  return FDVLM_OK;
}

extern "C" int fdvlm_block_step(fdvlm_t* h, const fdvlm_step_params* p, float* logits, float* conf, int32_t* pred,
                                uint8_t* unmask, int32_t* block_tokens, fdvlm_step_info* info) {
  int rc = step_core(h, p);
  if (rc) return rc;
  const int B = h->block_size;
  const cudaMemcpyKind DD = cudaMemcpyDeviceToDevice;
  if (logits) CU(h, cudaMemcpyAsync(logits, h->logits, (size_t)B * h->cfg.vocab * 4, DD, h->st));
  if (conf) CU(h, cudaMemcpyAsync(conf, h->conf, (size_t)B * 4, DD, h->st));
  if (pred) CU(h, cudaMemcpyAsync(pred, h->pred, (size_t)B * 4, DD, h->st));
  if (unmask) CU(h, cudaMemcpyAsync(unmask, h->unmask, (size_t)B, DD, h->st));
  if (block_tokens) CU(h, cudaMemcpyAsync(block_tokens, h->blk_tokens, (size_t)B * 4, DD, h->st));
  // the host needs n_remaining to police the state machine, so the read-back always happens
  return finish_info(h, info);
}

extern "C" int fdvlm_block_step_host(fdvlm_t* h, const fdvlm_step_params* p, float* conf_host, int32_t* pred_host,
                                     uint8_t* unmask_host, int32_t* block_tokens_host, fdvlm_step_info* info) {
  int rc = step_core(h, p);
  if (rc) return rc;
  const int B = h->block_size;
  char* s = h->host_stage;  // [conf 256 | pred 256 | tokens 256 | unmask 64]
  const cudaMemcpyKind DH = cudaMemcpyDeviceToHost;
  if (conf_host) CU(h, cudaMemcpyAsync(s, h->conf, (size_t)B * 4, DH, h->st));
  if (pred_host) CU(h, cudaMemcpyAsync(s + 256, h->pred, (size_t)B * 4, DH, h->st));
  if (block_tokens_host) CU(h, cudaMemcpyAsync(s + 512, h->blk_tokens, (size_t)B * 4, DH, h->st));
  if (unmask_host) CU(h, cudaMemcpyAsync(s + 768, h->unmask, (size_t)B, DH, h->st));
  rc = finish_info(h, info);
  if (rc) return rc;
  if (conf_host) memcpy(conf_host, s, (size_t)B * 4);
  if (pred_host) memcpy(pred_host, s + 256, (size_t)B * 4);
  if (block_tokens_host) memcpy(block_tokens_host, s + 512, (size_t)B * 4);
  if (unmask_host) memcpy(unmask_host, s + 768, (size_t)B);
  return FDVLM_OK;
}

extern "C" int fdvlm_commit_block(fdvlm_t* h, float* next_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "commit without an open block");
  if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "commit with %d masked positions left", h->n_remaining);
  const int B = h->block_size;
  h->launches = 0;
  launch_embed(h->w.embed, h->blk_tokens, h->h, B, h->cfg.hidden, h->dt == DT_F32 ? DT_F32 : DT_BF16, h->st);
  h->launches++;
  int rc = forward_rows(h, B, MODE_CAUSAL, next_logits ? 1 : 0);
  if (rc) return rc;
  if (next_logits) CU(h, cudaMemcpyAsync(next_logits, h->logits, (size_t)h->cfg.vocab * 4, cudaMemcpyDeviceToDevice, h->st));
  h->cache_len += B;
  h->block_open = 0;
  h->block_size = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_cache_read(const fdvlm_t* hc, int layer, int which, int pos0, int n, void* dst) {
  fdvlm_t* h = const_cast<fdvlm_t*>(hc);
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!dst || layer < 0 || layer >= h->cfg.n_layers || (which != 0 && which != 1) || pos0 < 0 || n < 0 ||
      pos0 + n > h->cfg.max_seq)
    return fail(h, FDVLM_ERR_INVALID_ARG, "cache_read: bad argument");
  const int d = h->cfg.head_dim, hkv = h->cfg.n_kv_heads;
  // cache plane is [Hkv][max_seq][d]; dst is [n][Hkv][d]
  const size_t rowb = (size_t)d * h->act_sz;
  for (int hk = 0; hk < hkv; ++hk) {
    const char* src = kv_ptr(h, layer, which) + ((size_t)hk * h->cfg.max_seq + pos0) * rowb;
    CU(h, cudaMemcpy2DAsync((char*)dst + hk * rowb, (size_t)hkv * rowb, src, rowb, rowb, (size_t)n, cudaMemcpyDeviceToDevice, h->st));
  }
  return FDVLM_OK;
}

// ---- instrumentation --------------------------------------------------------------------------------
extern "C" int fdvlm_profile_enable(fdvlm_t* h, int on) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  h->prof_on = on ? 1 : 0;
  h->prof_used = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_profile_read(fdvlm_t* h, double* ms_linear, int* n_linear, double* ms_attention, int* n_attention) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  CU(h, cudaStreamSynchronize(h->st));
  double ms[2] = {0, 0};
  int cnt[2] = {0, 0};
  for (size_t i = 0; i < h->prof_used; ++i) {
    float t = 0.f;
    CU(h, cudaEventElapsedTime(&t, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]));
    ms[h->prof_kind[i]] += t;
    cnt[h->prof_kind[i]]++;
  }
  if (ms_linear) *ms_linear = ms[0];
  if (n_linear) *n_linear = cnt[0];
  if (ms_attention) *ms_attention = ms[1];
  if (n_attention) *n_attention = cnt[1];
  h->prof_used = 0;
  return FDVLM_OK;
}

// ---- single operators ---------------------------------------------------------------------------------
extern "C" size_t fdvlm_op_linear_workspace_bytes(int m, int n, int k, fdvlm_dtype dtype) {
  if (m < 1 || n < 1 || k < 1) return 0;
  return linear_workspace_bytes(m, n, k, (int)dtype);
}

extern "C" int fdvlm_op_linear(const void* x, const void* w, const float* scale, const float* bias, float* y, int m,
                               int n, int k, fdvlm_dtype dtype, void* workspace, void* cuda_stream) {
  if (!x || !w || !y || m < 1 || m > 64 || n < 1 || k < 8 || (k % 8)) return FDVLM_ERR_INVALID_ARG;
  if (dtype != FDVLM_F32 && dtype != FDVLM_BF16 && dtype != FDVLM_W_FP8E4M3) return FDVLM_ERR_INVALID_ARG;
  if (dtype == FDVLM_W_FP8E4M3 && !scale) return FDVLM_ERR_INVALID_ARG;
  LinearArgs a;
  a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = n; a.k = k; a.ldy = n; a.accumulate = 0;
  a.dtype = (int)dtype; a.workspace = workspace; a.workspace_bytes = linear_workspace_bytes(m, n, k, (int)dtype);
  if (a.workspace_bytes && !workspace) return FDVLM_ERR_INVALID_ARG;
  cudaError_t e;
  int r = launch_linear(a, (cudaStream_t)cuda_stream, &e);
  return r < 0 ? FDVLM_ERR_CUDA : FDVLM_OK;
}

extern "C" size_t fdvlm_op_attention_workspace_bytes(int n_rows, int n_q_heads, int n_kv_heads, int head_dim) {
  return attention_workspace_bytes(n_rows, n_q_heads, n_kv_heads, head_dim);
}

extern "C" int fdvlm_op_attention(const void* q, const void* k_cache, const void* v_cache, void* out, int n_rows,
                                  int cache_len, int max_seq, int n_q_heads, int n_kv_heads, int head_dim, int causal,
                                  fdvlm_dtype dtype, void* workspace, void* cuda_stream) {
  if (!q || !k_cache || !v_cache || !out || n_rows < 1 || n_rows > 64 || cache_len < 0 || cache_len + n_rows > max_seq ||
      n_q_heads < 1 || n_kv_heads < 1 || (n_q_heads % n_kv_heads) || (head_dim != 64 && head_dim != 128))
    return FDVLM_ERR_INVALID_ARG;
  if (dtype != FDVLM_F32 && dtype != FDVLM_BF16 && dtype != FDVLM_W_FP8E4M3) return FDVLM_ERR_INVALID_ARG;
  AttnArgs a;
  a.q = q; a.kc = k_cache; a.vc = v_cache; a.out = out; a.n = n_rows; a.cache_len = cache_len; a.max_seq = max_seq;
  a.hq = n_q_heads; a.hkv = n_kv_heads; a.d = head_dim; a.causal = causal ? 1 : 0; a.dtype = (int)dtype; a.workspace = workspace;
  cudaError_t e;
  int r = launch_attention(a, (cudaStream_t)cuda_stream, &e);
  return r < 0 ? FDVLM_ERR_CUDA : FDVLM_OK;
}
