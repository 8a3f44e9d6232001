// The decoder forward of one step as a launch sequence (Fast-dVLM Sec. 3.4; Appendix B Alg. 1 for the
// two attention modes), in two flavours: the exact CUDA-core path (fp32 configuration, shapes the
// tensor-core kernels do not take) and the tensor-core path (bf16 and fp8 weights).
#include "handle.h"

namespace fdk {

int launch_linear_simt(const LinearArgs& a, cudaStream_t st, cudaError_t* err);
size_t simt_workspace_bytes(int m, int n, int k);
int launch_attention_simt(const AttnArgs& a, cudaStream_t st, cudaError_t* err);
size_t attention_mma_workspace_bytes(int n, int hq, int hkv, int d);
int launch_attention_mma(const AttnArgs& a, cudaStream_t st, cudaError_t* err);
void launch_splitk_epilogue(const float* part, int S, int m, int n, const float* scale, const float* bias, float* y, int ldy,
                            int accumulate, cudaStream_t st, const float* row_amax = nullptr);

thread_local char g_create_error[512] = "";

// Stand-alone projection.  The caller's workspace starts with OP_HEAD bytes for the two status words (see
// TcOut::status; cleared here on the stream), then -- fp8 weights only -- an f16 copy of the bf16 rows (W8A8: followed
// by one 256-byte-rounded array of per-row maxima), then the split-K partial sums.
static size_t op_amax_bytes(int m, int dtype) { return dtype == DT_A8 ? (((size_t)m * 4 + 255) / 256) * 256 : 0; }
static size_t op_x16_bytes(int m, int k, int dtype) {
  return (dtype == DT_FP8 || dtype == DT_A8) ? (((size_t)m * k * 2 + 255) / 256) * 256 + op_amax_bytes(m, dtype) : 0;
}
size_t linear_workspace_bytes(int m, int n, int k, int dtype) {
  const int wdt = dtype == DT_A8 ? DT_FP8 : dtype;
  size_t a = dtype == DT_A8 ? 0 : simt_workspace_bytes(m, n, k);
  size_t b = tc_linear_supported(m, n, k, wdt) ? tc_workspace_bytes(m, n, (n + 127) / 128, k) + op_x16_bytes(m, k, dtype) : 0;
  return OP_HEAD + (a > b ? a : b);
}

// One projection y = x w^T (* scale) (+ bias) (+ y): bf16 / fp8 weights go to the tensor-core kernel
// (split-K partial sums + fixed-order reduction), everything else to the CUDA-core kernel.
int launch_linear(const LinearArgs& a, cudaStream_t st, cudaError_t* err) {
  if (!a.workspace || a.workspace_bytes < OP_HEAD) { *err = cudaErrorInvalidValue; return -1; }
  *err = cudaMemsetAsync(a.workspace, 0, 8, st);
  if (*err != cudaSuccess) return -1;
  LinearArgs b = a;
  b.workspace = (char*)a.workspace + OP_HEAD;
  b.workspace_bytes = a.workspace_bytes - OP_HEAD;
  const bool a8 = a.dtype == DT_A8;
  if (!tc_linear_supported(a.m, a.n, a.k, a8 ? DT_FP8 : a.dtype)) {
    if (a8) { *err = cudaErrorNotSupported; return -1; }      // the quantising projection exists on the tensor cores only
    return launch_linear_simt(b, st, err);
  }
  TcGroup g;
  memset(&g, 0, sizeof(g));
  g.x = a.x; g.m = a.m; g.k = a.k; g.w[0] = a.w; g.n[0] = a.n; g.n_mats = 1;
  g.fp8 = (a.dtype == DT_FP8 || a8); g.a8 = a8;
  const size_t x16 = op_x16_bytes(a.m, a.k, a.dtype);
  if (b.workspace_bytes < x16) { *err = cudaErrorInvalidValue; return -1; }
  float* row_amax = a8 ? (float*)((char*)b.workspace + x16 - op_amax_bytes(a.m, a.dtype)) : nullptr;
  int launched = 2;
  if (a8) {        // f16 rows and each row's maximum: the kernel quantises the rows to e4m3 itself
    launch_bf16_rows_to_f16_amax(a.x, b.workspace, a.m, a.k, row_amax, st);
    g.x = b.workspace;
    ++launched;
  } else if (g.fp8) {     // the fp8 GEMM multiplies f16 by f16
    launch_bf16_to_f16(a.x, b.workspace, (size_t)a.m * a.k, st);
    g.x = b.workspace;
    ++launched;
  }
  float* part = (float*)((char*)b.workspace + x16);
  int splits = 0;
  TcOut o;
  memset(&o, 0, sizeof(o));
  o.mode = TC_MODE_PARTIAL; o.part = part; o.part_bytes = b.workspace_bytes - x16; o.splits_out = &splits;
  o.ld = a.n; o.status = (int*)a.workspace;
  o.amax_in = row_amax; o.n_amax_in = 1;
  *err = tc_group_launch(g, o, st);
  if (*err != cudaSuccess) return -1;
  launch_splitk_epilogue(part, splits, a.m, a.n, a.scale, a.bias, a.y, a.ldy, a.accumulate, st, row_amax);
  *err = cudaGetLastError();
  return *err == cudaSuccess ? launched : -1;
}

size_t attention_workspace_bytes(int n, int hq, int hkv, int d) { return attention_mma_workspace_bytes(n, hq, hkv, d); }
// 16-bit rows go to the split-KV tensor-core kernel, fp32 rows to the exact CUDA-core kernel.
int launch_attention(const AttnArgs& a, cudaStream_t st, cudaError_t* err) {
  return a.dtype == DT_F32 ? launch_attention_simt(a, st, err) : launch_attention_mma(a, st, err);
}

int stage_rows(fdvlm_t* h, int row0, int n, const int32_t* tokens, const void* embeds) {
  const int H = h->cfg.hidden;
  const int edt = h->dt == DT_F32 ? DT_F32 : DT_BF16;
  if (h->use_tc) {
    launch_embed_prep(h->w.embed, tokens, embeds, h->h + (size_t)row0 * H, (char*)h->a + (size_t)row0 * H * 2, h->a_lo, h->xfmt,
                      h->layers[0].g_attn, h->ssq + (size_t)row0 * h->nt, h->nt, n, H, h->cfg.vocab, h->info + 3, h->st, nullptr,
                      h->act8 ? h->amax_a + (size_t)row0 * h->nt : nullptr);
  } else if (tokens) {
    launch_embed(h->w.embed, tokens, h->h + (size_t)row0 * H, n, H, edt, h->cfg.vocab, h->info + 3, h->st);
  } else {
    launch_rows_to_f32(embeds, h->h + (size_t)row0 * H, n, H, edt, h->st);
  }
  h->launches++;
  CU(h, cudaGetLastError());
  return FDVLM_OK;
}

// ---- exact CUDA-core path: one kernel per operator ---------------------------------------------------
static int forward_rows_simt(fdvlm_t* h, int n, int mode, int logits_rows) {
  const fdvlm_config& c = h->cfg;
  const int H = c.hidden, I = c.intermediate, d = c.head_dim;
  const int NQ = c.n_q_heads * d, NKV = c.n_kv_heads * d, NQKV = NQ + 2 * NKV;
  cudaError_t e = cudaSuccess;
  auto lin = [&](const void* x, const void* w, const float* scale, const float* bias, float* y, int nn, int kk, int ldy,
                 int accumulate, int m, int dt) -> int {
    LinearArgs a;
    a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = nn; a.k = kk; a.ldy = ldy;
    a.accumulate = accumulate; a.dtype = dt; a.workspace = h->ws; a.workspace_bytes = h->ws_bytes;
    prof_begin(h, 0);
    int r = launch_linear_simt(a, h->st, &e);
    prof_end(h);
    if (r < 0) return -1;
    h->launches += r;
    return 0;
  };
  const int dt = h->dt;
  launch_rope_table(h->cs, n, h->cache_len, d, c.rope_theta, h->st, nullptr, nullptr, mode == MODE_MASKED ? h->q_pos_off : nullptr);
  h->launches++;
  for (int l = 0; l < c.n_layers; ++l) {
    const fdvlm_layer_weights& lw = h->layers[l];
    launch_rmsnorm(h->h, lw.g_attn, h->a, n, H, c.rms_eps, dt, h->st);
    if (lin(h->a, lw.wq, lw.s_q, lw.bq, h->y, NQ, H, NQKV, 0, n, dt) || lin(h->a, lw.wk, lw.s_k, lw.bk, h->y + NQ, NKV, H, NQKV, 0, n, dt) ||
        lin(h->a, lw.wv, lw.s_v, lw.bv, h->y + NQ + NKV, NKV, H, NQKV, 0, n, dt))
      return fail(h, FDVLM_ERR_CUDA, "qkv projection launch: %s", cudaGetErrorString(e));
    launch_qkv_post(h->y, h->cs, h->q, kv_ptr(h, l, 0), kv_ptr(h, l, 1), n, h->cache_len, c.n_q_heads, c.n_kv_heads, d,
                    c.max_seq, dt, h->st);
    AttnArgs at;
    memset(&at, 0, sizeof(at));
    at.q = h->q; at.kc = kv_ptr(h, l, 0); at.vc = kv_ptr(h, l, 1); at.out = h->ao; at.n = n; at.cache_len = h->cache_len;
    at.max_seq = c.max_seq; at.hq = c.n_q_heads; at.hkv = c.n_kv_heads; at.d = d; at.causal = (mode == MODE_CAUSAL);
    at.row_mask = (mode == MODE_MASKED) ? h->q_mask : (mode == MODE_FUSED ? h->f_mask : nullptr);
    at.dtype = dt; at.workspace = h->ws; at.kv_type = KV_BF16; at.out_fmt = XF_BF16; at.long_cache = -1;
    prof_begin(h, 1);
    int r = launch_attention(at, h->st, &e);
    prof_end(h);
    if (r < 0) return fail(h, FDVLM_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    h->launches += r + 2;
    if (lin(h->ao, lw.wo, lw.s_o, nullptr, h->h, H, NQ, H, 1, n, dt))
      return fail(h, FDVLM_ERR_CUDA, "o projection launch: %s", cudaGetErrorString(e));
    launch_rmsnorm(h->h, lw.g_mlp, h->a, n, H, c.rms_eps, dt, h->st);
    if (lin(h->a, lw.w_gate, lw.s_gate, nullptr, h->y, I, H, 2 * I, 0, n, dt) || lin(h->a, lw.w_up, lw.s_up, nullptr, h->y + I, I, H, 2 * I, 0, n, dt))
      return fail(h, FDVLM_ERR_CUDA, "gate/up projection launch: %s", cudaGetErrorString(e));
    launch_swiglu(h->y, h->act, n, I, dt, h->st);
    if (lin(h->act, lw.w_down, lw.s_down, nullptr, h->h, H, I, H, 1, n, dt))
      return fail(h, FDVLM_ERR_CUDA, "down projection launch: %s", cudaGetErrorString(e));
    h->launches += 2;
  }
  if (logits_rows > 0) {
    const int first = (logits_rows == n) ? 0 : n - 1;
    const int m = n - first;
    launch_rmsnorm(h->h + (size_t)first * H, h->w.g_final, h->a, m, H, c.rms_eps, dt, h->st);
    h->launches++;
    const void* table = c.tie_embeddings ? h->w.embed : h->w.lm_head;
    const float* sc = c.tie_embeddings ? nullptr : h->w.s_lm_head;
    // a tied table is stored in the embedding's type: fp32 for F32, bf16 otherwise (never fp8)
    const int hdt = (c.tie_embeddings && dt == DT_FP8) ? DT_BF16 : dt;
    if (lin(h->a, table, sc, nullptr, h->logits, c.vocab, H, c.vocab, 0, m, hdt))
      return fail(h, FDVLM_ERR_CUDA, "lm head launch: %s", cudaGetErrorString(e));
    if (logits_rows == n) {
      launch_row_stats(h->logits, n, c.vocab, c.mask_id, h->conf, h->pred, h->st);
      h->launches++;
    }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

// ---- tensor-core path (bf16 / fp8 weights) ---------------------------------------------------------------
// per layer: [QKV GEMM -> split-K partials] [sum + folded norm + bias + rotary + K/V staging] [attention + chunk merge]
//            [O GEMM -> partials] [sum + residual + gain + ssq] [gate/up GEMM, folded norm + SwiGLU epilogue]
//            [down GEMM -> partials] [sum + residual + gain + ssq]
// head:      [LM-head GEMM, folded final norm, logits + softmax statistics epilogue] [statistics merge]
// stamped: every launch gets the next record of h->stamps (in-chain timing, fdvlm_profile_enable(h, 2)).
static int forward_rows_tc(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits, const int* len_ptr, bool stamped,
                           int long_cache = -1) {
  const fdvlm_config& c = h->cfg;
  const int H = c.hidden, I = c.intermediate, d = c.head_dim, nt = h->nt;
  const int NQ = c.n_q_heads * d, NKV = c.n_kv_heads * d, NQKV = NQ + 2 * NKV;
  float* part = (float*)h->ws;
  cudaError_t e = cudaSuccess;
  if (stamped) { h->stamp_kind.clear(); h->stamp_used = 0; }
  auto stamp = [&](int kind) -> KStamp* {
    if (!stamped || h->stamp_used >= FDVLM_MAX_STAMPS) return nullptr;
    h->stamp_kind.push_back(kind);
    return h->stamps + h->stamp_used++;
  };
  const bool fp8 = (h->dt == DT_FP8);
  const bool a8 = h->act8 != 0;                      // W8A8: the four layer projections quantise their input rows
  // a GEMM input buffer: hi (or only) plane, and its lo plane when the format has one
  auto group = [&](const void* x, size_t lo_off, size_t row0_elems, int m, int k, int nm, const void* w0, int n0, const void* w1, int n1,
                   const void* w2, int n2) {
    TcGroup g;
    memset(&g, 0, sizeof(g));
    g.x = (const char*)x + row0_elems * 2; g.m = m; g.k = k; g.n_mats = nm;
    g.x_lo = (h->xfmt == XF_BF16X2) ? (const char*)x + (lo_off + row0_elems) * 2 : nullptr;
    g.w[0] = w0; g.n[0] = n0; g.w[1] = w1; g.n[1] = n1; g.w[2] = w2; g.n[2] = n2;
    g.fp8 = fp8; g.a8 = a8;
    return g;
  };
  auto out = [&](int tc_mode, int kind) {
    TcOut o;
    memset(&o, 0, sizeof(o));
    o.mode = tc_mode; o.status = h->info + 3; o.part = part; o.part_bytes = h->ws_bytes; o.stamp = stamp(kind);
    return o;
  };
  auto gemm = [&](const TcGroup& g, const TcOut& o) {
    prof_begin(h, 0);
    e = tc_group_launch(g, o, h->st);
    prof_end(h);
    h->launches++;
    return e == cudaSuccess;
  };
  launch_rope_table(h->cs, n, h->cache_len, d, c.rope_theta, h->st, len_ptr, stamp(FDVLM_K_ROPE_TABLE),
                    mode == MODE_MASKED ? h->q_pos_off : nullptr);
  h->launches++;
  for (int l = 0; l < c.n_layers; ++l) {
    const fdvlm_layer_weights& lw = h->layers[l];
    int S = 0;
    TcOut o = out(TC_MODE_PARTIAL, FDVLM_K_GEMM_QKV);
    o.ld = NQKV; o.splits_out = &S;
    o.amax_in = a8 ? h->amax_a : nullptr; o.n_amax_in = nt;
    if (!gemm(group(h->a, h->a_lo, 0, n, H, 3, lw.wq, NQ, lw.wk, NKV, lw.wv, NKV), o))
      return fail(h, FDVLM_ERR_CUDA, "qkv projection launch: %s", cudaGetErrorString(e));
    launch_fin_qkv(part, S, n, h->cs, h->ssq, nt, H, c.rms_eps, lw.bq, lw.bk, lw.bv, lw.s_q, lw.s_k, lw.s_v, h->q, kv_ptr(h, l, 0), kv_ptr(h, l, 1),
                   h->cache_len, c.n_q_heads, c.n_kv_heads, d, c.max_seq, h->kv_type, h->st, len_ptr, stamp(FDVLM_K_FIN_QKV),
                   a8 ? h->amax_a : nullptr, a8 ? h->amax_act : nullptr);
    AttnArgs at;
    memset(&at, 0, sizeof(at));
    at.len_ptr = len_ptr;
    at.q = h->q; at.kc = kv_ptr(h, l, 0); at.vc = kv_ptr(h, l, 1); at.out = h->ao; at.n = n; at.cache_len = h->cache_len;
    at.max_seq = c.max_seq; at.hq = c.n_q_heads; at.hkv = c.n_kv_heads; at.d = d; at.causal = (mode == MODE_CAUSAL);
    at.row_mask = (mode == MODE_MASKED) ? h->q_mask : (mode == MODE_FUSED ? h->f_mask : nullptr);
    at.dtype = h->dt; at.workspace = h->ws; at.kv_type = h->kv_type; at.out_fmt = h->xfmt; at.out_lo_off = h->ao_lo;
    at.status = h->info + 3;
    at.amax_out = a8 ? h->amax_ao : nullptr;
    at.long_cache = long_cache;
    at.stamp = stamp(FDVLM_K_ATTENTION);
    if (at.stamp && !stamp(FDVLM_K_ATTN_MERGE)) at.stamp = nullptr;     // the launcher uses two consecutive records
    prof_begin(h, 1);
    int r = launch_attention(at, h->st, &e);
    prof_end(h);
    if (r < 0) return fail(h, FDVLM_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    h->launches += r + 1;
    o = out(TC_MODE_PARTIAL, FDVLM_K_GEMM_O);
    o.ld = H; o.splits_out = &S;
    o.amax_in = a8 ? h->amax_ao : nullptr; o.n_amax_in = c.n_q_heads;
    if (!gemm(group(h->ao, h->ao_lo, 0, n, NQ, 1, lw.wo, H, nullptr, 0, nullptr, 0), o))
      return fail(h, FDVLM_ERR_CUDA, "o projection launch: %s", cudaGetErrorString(e));
    launch_fin_resid(part, S, n, H, h->h, lw.g_mlp, h->a, h->a_lo, h->xfmt, h->ssq, nt, lw.s_o, h->st, stamp(FDVLM_K_FIN_RESID),
                     a8 ? h->amax_ao : nullptr, c.n_q_heads, a8 ? h->amax_a : nullptr);
    o = out(TC_MODE_SWIGLU, FDVLM_K_GEMM_GATE_UP);
    o.act = h->act; o.act_lo_off = h->act_lo; o.act_fmt = h->xfmt;
    o.ssq_in = h->ssq; o.nt_in = nt; o.hidden = H; o.eps = c.rms_eps;
    o.amax_in = a8 ? h->amax_a : nullptr; o.n_amax_in = nt; o.amax_out = a8 ? h->amax_act : nullptr;
    TcGroup gu = group(h->a, h->a_lo, 0, n, H, 2, lw.w_gate, I, lw.w_up, I, nullptr, 0);
    gu.scale[0] = lw.s_gate; gu.scale[1] = lw.s_up;
    if (!gemm(gu, o))
      return fail(h, FDVLM_ERR_CUDA, "gate/up projection launch: %s", cudaGetErrorString(e));
    o = out(TC_MODE_PARTIAL, FDVLM_K_GEMM_DOWN);
    o.ld = H; o.splits_out = &S;
    o.amax_in = a8 ? h->amax_act : nullptr; o.n_amax_in = 1;
    if (!gemm(group(h->act, h->act_lo, 0, n, I, 1, lw.w_down, H, nullptr, 0, nullptr, 0), o))
      return fail(h, FDVLM_ERR_CUDA, "down projection launch: %s", cudaGetErrorString(e));
    // the last layer feeds the LM head, whose table (a tied bf16 embedding under fp8 layer weights) may want another format
    const bool last = (l + 1 == c.n_layers);
    const float* g_next = last ? h->w.g_final : h->layers[l + 1].g_attn;
    launch_fin_resid(part, S, n, H, h->h, g_next, h->a, h->a_lo, last ? h->head_fmt : h->xfmt, h->ssq, nt, lw.s_down, h->st,
                     stamp(FDVLM_K_FIN_RESID), a8 ? h->amax_act : nullptr, 1, (a8 && !last) ? h->amax_a : nullptr);
    h->launches += 2;
  }
  if (logits_rows > 0) {
    const int first = (logits_rows == n) ? 0 : n - 1;
    const int m = n - first;
    const void* table = c.tie_embeddings ? h->w.embed : h->w.lm_head;
    TcOut o = out(TC_MODE_LOGITS, FDVLM_K_GEMM_LM_HEAD);
    o.y = h->logits; o.ld = c.vocab; o.write_logits = (logits_rows == n) ? want_logits : 1;
    o.ssq_in = h->ssq + (size_t)first * nt; o.nt_in = nt; o.hidden = H; o.eps = c.rms_eps;
    o.stats = h->stats; o.mask_id = c.mask_id;
    TcGroup lm = group(h->a, h->a_lo, (size_t)first * H, m, H, 1, table, c.vocab, nullptr, 0, nullptr, 0);
    lm.fp8 = (h->head_fmt == XF_F16);
    lm.a8 = 0;                                       // the LM head keeps 16-bit input rows
    lm.x_lo = (h->head_fmt == XF_BF16X2) ? (const char*)h->a + (h->a_lo + (size_t)first * H) * 2 : nullptr;
    if (!c.tie_embeddings) lm.scale[0] = h->w.s_lm_head;
    if (!gemm(lm, o))
      return fail(h, FDVLM_ERR_CUDA, "lm head launch: %s", cudaGetErrorString(e));
    if (logits_rows == n) {
      launch_stats_merge(h->stats, ceil_div(c.vocab, 128) * 4, n, h->conf, h->pred, h->st, stamp(FDVLM_K_STATS_MERGE));
      h->launches++;
    }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

// The tensor-core forward as a replayed CUDA graph: every kernel takes the cache length from a device word, so one
// capture per (rows, mode, logits mode, stamped or not) serves every later call; the programmatic-dependent-launch
// edges are kept.
static int forward_rows_graph(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits) {
  const int stamped = (h->prof_on == 2) ? 1 : 0;
  const int long_cache = attention_long_cache(h->cache_len + n) ? 1 : 0;
  launch_set_len(h->dev_len, h->cache_len, h->st);
  h->launches++;
  if (stamped) CU(h, cudaMemsetAsync(h->stamps, 0xFF, sizeof(KStamp) * FDVLM_MAX_STAMPS, h->st));
  for (auto& g : h->graphs) {
    if (g.n == n && g.mode == mode && g.logits_rows == logits_rows && g.want_logits == want_logits && g.stamped == stamped &&
        g.long_cache == long_cache) {
      if (stamped) {      // the records' kinds are those of the capture: replay the bookkeeping only
        h->stamp_kind = g.kinds;
        h->stamp_used = (int)g.kinds.size();
      }
      CU(h, cudaGraphLaunch(g.exec, h->st));
      h->launches += g.launches;
      return FDVLM_OK;
    }
  }
  const int before = h->launches;
  CU(h, cudaStreamBeginCapture(h->st, cudaStreamCaptureModeThreadLocal));
  const int rc = forward_rows_tc(h, n, mode, logits_rows, want_logits, h->dev_len, stamped != 0, long_cache);
  cudaGraph_t graph = nullptr;
  cudaError_t e = cudaStreamEndCapture(h->st, &graph);
  if (rc != FDVLM_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "graph capture: %s", cudaGetErrorString(e));
  fdvlm::FwdGraph g;
  g.n = n; g.mode = mode; g.logits_rows = logits_rows; g.want_logits = want_logits; g.stamped = stamped; g.long_cache = long_cache;
  g.launches = h->launches - before; g.exec = nullptr;
  if (stamped) g.kinds = h->stamp_kind;
  e = cudaGraphInstantiate(&g.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "graph instantiate: %s", cudaGetErrorString(e));
  h->graphs.push_back(g);
  CU(h, cudaGraphLaunch(g.exec, h->st));
  return FDVLM_OK;
}

// The kernels of one tensor-core forward enqueued on the handle's stream, cache length taken from the device word:
// what a caller that is itself capturing the stream (the on-device decode loop) records.
int forward_rows_enqueue(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits) {
  return forward_rows_tc(h, n, mode, logits_rows, want_logits, h->dev_len, false, attention_long_cache(h->cache_len + n) ? 1 : 0);
}

int forward_rows(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits) {
  if (!h->use_tc) return forward_rows_simt(h, n, mode, logits_rows);
  // event timing around each kernel needs the kernels launched one by one
  if (h->use_graphs && h->prof_on != 1) return forward_rows_graph(h, n, mode, logits_rows, want_logits);
  const bool stamped = h->prof_on == 2;
  if (stamped) CU(h, cudaMemsetAsync(h->stamps, 0xFF, sizeof(KStamp) * FDVLM_MAX_STAMPS, h->st));
  return forward_rows_tc(h, n, mode, logits_rows, want_logits, nullptr, stamped);
}

}  // namespace fdk
