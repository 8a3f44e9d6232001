// The C ABI: handle life cycle, argument and state checks, and the request-level operations
// (Fast-dVLM Sec. 3.4 decode loop: prefill, block begin / step / commit).
#include <stdlib.h>

#include <new>

#include "handle.h"

using namespace fdk;

static int check_config(const fdvlm_config* c) {
  if (c->n_layers < 1 || c->hidden < 8 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->intermediate < 8 || c->vocab < 2)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "config: non-positive dimension");
  if (c->head_dim != 64 && c->head_dim != 128) return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (c->n_q_heads % c->n_kv_heads) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "n_q_heads not a multiple of n_kv_heads");
  if (c->dtype != FDVLM_F32 && c->dtype != FDVLM_BF16 && c->dtype != FDVLM_W_FP8E4M3 && c->dtype != FDVLM_W8A8_FP8E4M3)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "unknown dtype %d", (int)c->dtype);
  int mult = c->dtype == FDVLM_F32 ? 8 : 16;
  if (c->hidden % mult || c->intermediate % mult)
    return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "hidden and intermediate must be multiples of %d", mult);
  if (c->mask_id < 0 || c->mask_id >= c->vocab) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "mask_id out of range");
  if (c->max_block < 1 || c->max_block > 64) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "max_block must be in 1..64");
  if (c->max_seq < c->max_block) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "max_seq smaller than max_block");
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 0.f)) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "rms_eps / rope_theta must be positive");
  if (c->kv_dtype != FDVLM_KV_BF16 && c->kv_dtype != FDVLM_KV_F16) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "unknown kv_dtype %d", (int)c->kv_dtype);
  return FDVLM_OK;
}

extern "C" const char* fdvlm_version(void) { return "fdvlm 0.3 (sm_100a)"; }

extern "C" const char* fdvlm_last_error(const fdvlm_t* h) { return h ? h->err : g_create_error; }

extern "C" void fdvlm_destroy(fdvlm_t* h) {
  if (!h) return;
  for (auto& g : h->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
  h->graphs.clear();
  if (h->loop_exec) cudaGraphExecDestroy(h->loop_exec);
  if (h->kv) cudaFree(h->kv);
  if (h->slab) cudaFree(h->slab);
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
  const bool w8 = cfg->dtype == FDVLM_W_FP8E4M3 || cfg->dtype == FDVLM_W8A8_FP8E4M3;
  if (w8 && !cfg->tie_embeddings && !w->s_lm_head)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "fp8 lm_head needs s_lm_head");
  for (int l = 0; l < cfg->n_layers; ++l) {
    const fdvlm_layer_weights& lw = w->layers[l];
    if (!lw.wq || !lw.wk || !lw.wv || !lw.wo || !lw.w_gate || !lw.w_up || !lw.w_down || !lw.g_attn || !lw.g_mlp)
      return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: NULL weight", l);
    int nb = (lw.bq != nullptr) + (lw.bk != nullptr) + (lw.bv != nullptr);
    if (nb != 0 && nb != 3) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: biases must be all NULL or all set", l);
    if (w8 && (!lw.s_q || !lw.s_k || !lw.s_v || !lw.s_o || !lw.s_gate || !lw.s_up || !lw.s_down))
      return fail(nullptr, FDVLM_ERR_INVALID_ARG, "layer %d: fp8 weights need all scales", l);
  }
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev == 0) return fail(nullptr, FDVLM_ERR_CUDA, "no usable CUDA device: %s", cudaGetErrorString(e));

  fdvlm_t* h = new (std::nothrow) fdvlm;
  if (!h) return fail(nullptr, FDVLM_ERR_OOM, "host allocation failed");
  h->cfg = *cfg;
  h->layers.assign(w->layers, w->layers + cfg->n_layers);
  h->w = *w;
  h->w.layers = h->layers.data();
  h->st = (cudaStream_t)cuda_stream;
  h->act8 = cfg->dtype == FDVLM_W8A8_FP8E4M3 ? 1 : 0;       // W8A8 = the fp8-weight path with quantised projection inputs
  h->dt = h->act8 ? DT_FP8 : (int)cfg->dtype;
  h->act_sz = cfg->dtype == FDVLM_F32 ? 4 : 2;
  h->err[0] = 0;
  h->cache_len = h->block_size = h->n_remaining = h->step_index = h->block_open = 0;
  h->launches = 0;
  h->prof_on = 0;
  h->prof_used = 0;
  h->kv = nullptr; h->h = nullptr; h->a = h->ao = h->act = h->q = nullptr; h->y = nullptr; h->cs = nullptr; h->ssq = nullptr;
  h->amax_a = h->amax_ao = h->amax_act = nullptr;
  h->stats = nullptr; h->logits = nullptr; h->conf = nullptr; h->pred = nullptr; h->unmask = nullptr; h->blk_tokens = nullptr;
  h->blk_masked = nullptr; h->info = nullptr; h->init_stage = nullptr; h->ws = nullptr; h->info_host = nullptr;
  h->host_stage = nullptr;
  h->slab = nullptr;
  h->dev_len = nullptr;
  h->use_graphs = 0;
  h->stamps = nullptr;
  h->stamp_used = 0;
  h->loop_exec = nullptr;
  h->q_d = nullptr; h->q_mask = nullptr; h->q_pos_off = nullptr; h->quad_B = 0;
  h->f_rows = nullptr; h->f_mask = nullptr;
  cudaGetDevice(&h->device);

  const int R = cfg->max_block, H = cfg->hidden, I = cfg->intermediate, d = cfg->head_dim;
  const int NQ = cfg->n_q_heads * d, NKV = cfg->n_kv_heads * d, NQKV = NQ + 2 * NKV;
  h->nt = (H + 127) / 128;
  size_t ws = 0;
  const int shapes[][2] = {{NQ, H}, {NKV, H}, {H, NQ}, {I, H}, {H, I}, {cfg->vocab, H}};
  for (auto& s : shapes) { size_t b = linear_workspace_bytes(R, s[0], s[1], h->dt); if (b > ws) ws = b; }
  size_t wa = attention_workspace_bytes(R, cfg->n_q_heads, cfg->n_kv_heads, d);
  if (wa > ws) ws = wa;
  h->use_tc = (h->dt == DT_BF16 || h->dt == DT_FP8) && tc_linear_supported(R, NQ, H, h->dt) && tc_linear_supported(R, H, I, h->dt);
  h->kv_type = (int)cfg->kv_dtype;
  if (h->act8 && !h->use_tc) {
    delete h;
    return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "W8A8 needs shapes the tensor-core kernels take");
  }
  if (!h->use_tc && h->dt != DT_F32 && h->kv_type != KV_BF16) {
    delete h;
    return fail(nullptr, FDVLM_ERR_UNSUPPORTED, "an f16 KV cache needs shapes the tensor-core kernels take");
  }
  // GEMM inputs: bf16 hi + lo planes for bf16 weights, one f16 plane for fp8 weights (CUDA-core path: one plane)
  h->xfmt = !h->use_tc ? XF_BF16 : (h->dt == DT_FP8 ? XF_F16 : XF_BF16X2);
  h->head_fmt = (h->xfmt == XF_F16 && cfg->tie_embeddings) ? XF_BF16X2 : h->xfmt;
  const int planes = h->xfmt == XF_BF16X2 ? 2 : 1;
  const int a_planes = (h->xfmt == XF_BF16X2 || h->head_fmt == XF_BF16X2) ? 2 : 1;
  h->a_lo = (size_t)R * H; h->ao_lo = (size_t)R * NQ; h->act_lo = (size_t)R * I;
  if (h->use_tc) {
    const size_t g3[] = {tc_workspace_bytes(R, NQKV, (NQ + 127) / 128 + 2 * ((NKV + 127) / 128), H),
                         tc_workspace_bytes(R, H, (H + 127) / 128, NQ), tc_workspace_bytes(R, H, (H + 127) / 128, I)};
    for (size_t b : g3) if (b > ws) ws = b;
  }
  h->ws_bytes = ws;
  // Every buffer but the KV cache is carved out of one slab, the small hot ones first: with gigabytes of weights
  // streaming through the TLBs, each separately allocated buffer would cost its own page walk whenever it is touched.
  struct { void** p; size_t bytes; } allocs[] = {
      {(void**)&h->info, 32},
      {(void**)&h->dev_len, 16},
      {(void**)&h->conf, (size_t)R * 4},
      {(void**)&h->pred, (size_t)R * 4},
      {(void**)&h->unmask, 64},
      {(void**)&h->blk_tokens, 64 * 4},
      {(void**)&h->blk_masked, 64},
      {(void**)&h->init_stage, 64 * 4},
      {(void**)&h->q_d, 64 * 4},
      {(void**)&h->q_mask, 64 * 8},
      {(void**)&h->q_pos_off, 64 * 4},
      {(void**)&h->f_rows, 64 * 4},
      {(void**)&h->f_mask, 64 * 8},
      {(void**)&h->ssq, (size_t)R * h->nt * 4},
      {(void**)&h->amax_a, h->act8 ? (size_t)R * h->nt * 4 : 16},
      {(void**)&h->amax_ao, h->act8 ? (size_t)R * cfg->n_q_heads * 4 : 16},
      {(void**)&h->amax_act, h->act8 ? (size_t)R * 4 : 16},
      {(void**)&h->cs, (size_t)R * d * 4},
      {(void**)&h->stamps, h->use_tc ? sizeof(KStamp) * FDVLM_MAX_STAMPS : 16},
      {(void**)&h->h, (size_t)R * H * 4},
      {(void**)&h->a, (size_t)R * H * h->act_sz * a_planes},
      {(void**)&h->ao, (size_t)R * NQ * h->act_sz * planes},
      {(void**)&h->q, (size_t)R * NQ * h->act_sz},
      {(void**)&h->act, (size_t)R * I * h->act_sz * planes},
      {(void**)&h->stats, (size_t)((cfg->vocab + 127) / 128) * 4 * R * 16},
      {(void**)&h->y, (size_t)R * (NQKV > 2 * I ? NQKV : 2 * I) * 4},
      {(void**)&h->ws, ws ? ws : 16},
      {(void**)&h->logits, (size_t)R * cfg->vocab * 4},
  };
  size_t slab_bytes = 0;
  for (auto& a : allocs) slab_bytes += (a.bytes + 255) / 256 * 256;
  e = cudaMalloc((void**)&h->slab, slab_bytes);
  if (e == cudaSuccess) e = cudaMalloc((void**)&h->kv, (size_t)cfg->n_layers * 2 * kv_plane(h));
  if (e != cudaSuccess) {
    fail(nullptr, FDVLM_ERR_OOM, "cudaMalloc of the work buffers (%zu bytes) or the KV cache failed: %s", slab_bytes, cudaGetErrorString(e));
    cudaGetLastError();
    fdvlm_destroy(h);
    return FDVLM_ERR_OOM;
  }
  {
    char* cur = h->slab;
    for (auto& a : allocs) { *a.p = cur; cur += (a.bytes + 255) / 256 * 256; }
  }
  if (cudaMallocHost((void**)&h->info_host, 32) != cudaSuccess || cudaMallocHost((void**)&h->host_stage, 64 * 16) != cudaSuccess) {
    fail(nullptr, FDVLM_ERR_OOM, "pinned host allocation failed");
    fdvlm_destroy(h);
    return FDVLM_ERR_OOM;
  }
  e = cudaMemsetAsync(h->kv, 0, (size_t)cfg->n_layers * 2 * kv_plane(h), h->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->info, 0, 32, h->st);
  if (e != cudaSuccess) {
    fail(nullptr, FDVLM_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
    fdvlm_destroy(h);
    return FDVLM_ERR_CUDA;
  }
  // the tensor-core forward is replayed from captured CUDA graphs (FDVLM_NO_GRAPH=1: launch kernel by kernel)
  const char* no_graph = getenv("FDVLM_NO_GRAPH");
  // (the legacy default stream cannot be captured: a handle created on it launches kernel by kernel)
  h->use_graphs = h->use_tc && h->st != nullptr && !(no_graph && no_graph[0] == '1');
  *out = h;
  return FDVLM_OK;
}

extern "C" int fdvlm_reset(fdvlm_t* h) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  h->cache_len = 0;
  h->block_open = 0;
  h->quad_B = 0;
  h->block_size = h->n_remaining = h->step_index = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_cache_len(const fdvlm_t* h) { return h ? h->cache_len : (int)FDVLM_ERR_INVALID_ARG; }
extern "C" int fdvlm_last_launch_count(const fdvlm_t* h) { return h ? h->launches : (int)FDVLM_ERR_INVALID_ARG; }

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
    const int n = total - done < R ? total - done : R;
    int ne = 0;   // rows [done, done + n): embedding rows first, then token rows
    int rc;
    if (done < n_embeds) {
      ne = n_embeds - done < n ? n_embeds - done : n;
      rc = stage_rows(h, 0, ne, nullptr, (const char*)embeds + (size_t)done * H * h->act_sz);
      if (rc) return rc;
    }
    if (ne < n) {
      rc = stage_rows(h, ne, n - ne, tokens + (done + ne - n_embeds), nullptr);
      if (rc) return rc;
    }
    const bool last = (done + n == total);
    rc = forward_rows(h, n, MODE_CAUSAL, (last && last_logits) ? 1 : 0, 1);
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

// Read the 16-byte device record back: counts for the state machine, and the kernels' timeout word.
static int sync_info(fdvlm_t* h) {
  CU(h, cudaMemcpyAsync(h->info_host, h->info, 32, cudaMemcpyDeviceToHost, h->st));
  CU(h, cudaStreamSynchronize(h->st));
  h->n_remaining = h->info_host[1];
  if (h->info_host[3] != 0) {
    const int code = h->info_host[3];
    cudaMemsetAsync(h->info + 3, 0, 4, h->st);
    if (code == ST_BAD_TOKEN)
      return fail(h, FDVLM_ERR_INVALID_ARG, "a token id outside [0, %d) was given; token 0 was embedded in its place", h->cfg.vocab);
    return fail(h, FDVLM_ERR_TIMEOUT, "a bounded device-side wait gave up (kernel role %d); results of this call are invalid", code);
  }
  return FDVLM_OK;
}

extern "C" int fdvlm_synchronize(fdvlm_t* h) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  const int keep = h->n_remaining;        // the block state the host tracks is not this call's business
  const int rc = sync_info(h);
  h->n_remaining = keep;
  return rc;
}

extern "C" int fdvlm_debug_poison(fdvlm_t* h, int on) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  int32_t* stage = (int32_t*)(h->host_stage + 960);      // pinned, beyond what the *_host variants use
  CU(h, cudaStreamSynchronize(h->st));                   // an earlier value may still be in flight from the same slot
  *stage = on ? 1 : 0;
  CU(h, cudaMemcpyAsync(h->info + 4, stage, 4, cudaMemcpyHostToDevice, h->st));
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

static int check_step_params(fdvlm_t* h, const fdvlm_step_params* p) {
  if (!p) return fail(h, FDVLM_ERR_INVALID_ARG, "NULL step params");
  if (p->rule != FDVLM_RULE_THRESHOLD && p->rule != FDVLM_RULE_TOPK) return fail(h, FDVLM_ERR_INVALID_ARG, "unknown rule");
  if (p->rule == FDVLM_RULE_TOPK && p->k < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "top-k needs k >= 1");
  if (p->rule == FDVLM_RULE_THRESHOLD && !(p->threshold == p->threshold)) return fail(h, FDVLM_ERR_INVALID_ARG, "threshold is NaN");
  if (p->pred_shift != 0 && p->pred_shift != 1) return fail(h, FDVLM_ERR_INVALID_ARG, "pred_shift is 0 or 1");
  return FDVLM_OK;
}

static int step_core(fdvlm_t* h, const fdvlm_step_params* p, int want_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  int prc = check_step_params(h, p);
  if (prc) return prc;
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "block_step without an open block");
  if (h->n_remaining == 0) return fail(h, FDVLM_ERR_STATE, "block_step with no masked position left");
  const int B = h->block_size;
  h->launches = 0;
  int rc = stage_rows(h, 0, B, h->blk_tokens, nullptr);
  if (rc) return rc;
  rc = forward_rows(h, B, MODE_BIDIR, B, want_logits);
  if (rc) return rc;
  launch_select(h->conf, h->pred, h->blk_tokens, h->blk_masked, h->unmask, h->info, B, (int)p->rule, p->threshold, p->k, h->st,
                p->pred_shift);
  h->launches++;
  CU(h, cudaGetLastError());
  h->step_index++;
  return FDVLM_OK;
}

static int finish_info(fdvlm_t* h, fdvlm_step_info* info) {
  int rc = sync_info(h);
  if (rc) return rc;
  if (info) { info->n_unmasked = h->info_host[0]; info->n_remaining = h->info_host[1]; info->step_index = h->info_host[2]; }
  if (h->info_host[0] == 0 && h->info_host[1] > 0)
    return fail(h, FDVLM_ERR_STATE, "no position could be revealed: with pred_shift = 1 position 0 of the block must be a given token");
  return FDVLM_OK;
}

extern "C" int fdvlm_block_step(fdvlm_t* h, const fdvlm_step_params* p, float* logits, float* conf, int32_t* pred,
                                uint8_t* unmask, int32_t* block_tokens, fdvlm_step_info* info) {
  int rc = step_core(h, p, logits != nullptr);
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

extern "C" int fdvlm_decode_block_topk(fdvlm_t* h, int block_size, const int32_t* init_tokens, int k, int pred_shift,
                                       int32_t* block_tokens, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "decode_block_topk needs the host info struct");
  if (k < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "top-k needs k >= 1");
  int rc = fdvlm_block_begin(h, block_size, init_tokens);      // (reads the masked count back when tokens are given)
  if (rc) return rc;
  fdvlm_step_params p;
  p.rule = FDVLM_RULE_TOPK; p.threshold = 0.f; p.k = k; p.pred_shift = pred_shift;
  const int steps = (h->n_remaining + k - 1) / k;
  int launches = 0;
  for (int s = 0; s < steps; ++s) {
    h->n_remaining = 1;            // the device keeps the true count; the host checks it once, below
    rc = step_core(h, &p, 0);
    if (rc) return rc;
    launches += h->launches;
  }
  h->launches = launches;
  if (block_tokens) CU(h, cudaMemcpyAsync(block_tokens, h->blk_tokens, (size_t)block_size * 4, cudaMemcpyDeviceToDevice, h->st));
  rc = sync_info(h);
  if (rc) return rc;
  info->n_unmasked = h->info_host[0]; info->n_remaining = h->info_host[1]; info->step_index = h->info_host[2];
  if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "%d masked positions left after %d top-%d steps", h->n_remaining, steps, k);
  return FDVLM_OK;
}

// The decode loop of one block as a CUDA graph: a conditional WHILE node whose body is one denoise step (embedding
// of the block's tokens, the forward, the selection); the selection kernel sets the loop condition on the device.
// Built once per (block size, step parameters) and kept.  Dependent-launch edges are tried first; if the runtime
// refuses them inside a conditional body the kernels are recorded with ordinary edges.
static int decode_loop_rest(fdvlm_t* h, int block_size, const fdvlm_step_params* p, int32_t* block_tokens, fdvlm_step_info* info,
                            int steps_done);

static int build_loop_graph(fdvlm_t* h, int B, const fdvlm_step_params* p, bool with_pdl) {
  cudaGraph_t g = nullptr;
  CU(h, cudaGraphCreate(&g, 0));
  int rc = FDVLM_OK;
  cudaGraphExec_t exec = nullptr;
  int body_launches = 0;
  do {
    cudaGraphConditionalHandle cond;
    cudaError_t e = cudaGraphConditionalHandleCreate(&cond, g, 1, cudaGraphCondAssignDefault);
    if (e != cudaSuccess) { rc = fail(h, FDVLM_ERR_CUDA, "conditional handle: %s", cudaGetErrorString(e)); break; }
    cudaGraphNodeParams np = {cudaGraphNodeTypeConditional};
    np.type = cudaGraphNodeTypeConditional;
    np.conditional.handle = cond;
    np.conditional.type = cudaGraphCondTypeWhile;
    np.conditional.size = 1;
    cudaGraphNode_t node;
    e = cudaGraphAddNode(&node, g, nullptr, 0, &np);
    if (e != cudaSuccess) { rc = fail(h, FDVLM_ERR_CUDA, "conditional node: %s", cudaGetErrorString(e)); break; }
    cudaGraph_t body = np.conditional.phGraph_out[0];
    e = cudaStreamBeginCaptureToGraph(h->st, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { rc = fail(h, FDVLM_ERR_CUDA, "capture of the loop body: %s", cudaGetErrorString(e)); break; }
    pdl_disabled() = !with_pdl;
    const int before = h->launches;
    rc = stage_rows(h, 0, B, h->blk_tokens, nullptr);
    if (rc == FDVLM_OK) rc = forward_rows_enqueue(h, B, MODE_BIDIR, B, 0);
    if (rc == FDVLM_OK) {
      launch_select(h->conf, h->pred, h->blk_tokens, h->blk_masked, h->unmask, h->info, B, (int)p->rule, p->threshold, p->k, h->st,
                    p->pred_shift, cond, 1);
      h->launches++;
    }
    pdl_disabled() = false;
    body_launches = h->launches - before;
    cudaGraph_t captured = nullptr;
    e = cudaStreamEndCapture(h->st, &captured);
    if (rc != FDVLM_OK) break;
    if (e != cudaSuccess) { rc = fail(h, FDVLM_ERR_CUDA, "capture of the loop body: %s", cudaGetErrorString(e)); break; }
    e = cudaGraphInstantiate(&exec, g, 0);
    if (e != cudaSuccess) { rc = fail(h, FDVLM_ERR_CUDA, "instantiate of the loop graph: %s", cudaGetErrorString(e)); break; }
  } while (0);
  cudaGraphDestroy(g);
  if (rc != FDVLM_OK) { cudaGetLastError(); return rc; }
  if (h->loop_exec) cudaGraphExecDestroy(h->loop_exec);
  h->loop_exec = exec;
  h->loop_n = B; h->loop_rule = (int)p->rule; h->loop_k = p->k; h->loop_shift = p->pred_shift; h->loop_threshold = p->threshold;
  h->loop_body_launches = body_launches;
  h->loop_long = attention_long_cache(h->cache_len + B) ? 1 : 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_decode_block(fdvlm_t* h, int block_size, const int32_t* init_tokens, const fdvlm_step_params* p,
                                  int32_t* block_tokens, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "decode_block needs the host info struct");
  int rc = check_step_params(h, p);
  if (rc) return rc;
  if (!h->use_graphs) return fail(h, FDVLM_ERR_UNSUPPORTED, "decode_block needs the tensor-core path on a non-default stream");
  rc = fdvlm_block_begin(h, block_size, init_tokens);      // (reads the masked count back when tokens are given)
  if (rc) return rc;
  h->launches = 0;
  return decode_loop_rest(h, block_size, p, block_tokens, info, 0);
}

// The on-device loop over the open block's remaining denoise steps; steps_done of them have already run.
static int decode_loop_rest(fdvlm_t* h, int block_size, const fdvlm_step_params* p, int32_t* block_tokens, fdvlm_step_info* info,
                            int steps_done) {
  int rc = FDVLM_OK;
  const int first_launches = h->launches;
  if (h->n_remaining > 0) {
    const int long_cache = attention_long_cache(h->cache_len + block_size) ? 1 : 0;
    const bool have = h->loop_exec && h->loop_n == block_size && h->loop_rule == (int)p->rule && h->loop_k == p->k &&
                      h->loop_shift == p->pred_shift && h->loop_threshold == p->threshold && h->loop_long == long_cache;
    if (!have) {
      rc = build_loop_graph(h, block_size, p, true);
      if (rc) rc = build_loop_graph(h, block_size, p, false);
      if (rc) return rc;
    }
    launch_set_len(h->dev_len, h->cache_len, h->st);
    CU(h, cudaMemcpyAsync(h->info + 5, &steps_done, 4, cudaMemcpyHostToDevice, h->st));
    CU(h, cudaGraphLaunch(h->loop_exec, h->st));
  } else {
    CU(h, cudaMemcpyAsync(h->info + 5, &steps_done, 4, cudaMemcpyHostToDevice, h->st));
  }
  if (block_tokens) CU(h, cudaMemcpyAsync(block_tokens, h->blk_tokens, (size_t)block_size * 4, cudaMemcpyDeviceToDevice, h->st));
  rc = sync_info(h);
  if (rc) return rc;
  info->n_unmasked = h->info_host[0]; info->n_remaining = h->info_host[1]; info->step_index = h->info_host[2];
  h->step_index = h->info_host[2];
  h->launches = first_launches + 1 + (h->info_host[5] - steps_done) * h->loop_body_launches;
  if (h->n_remaining != 0)
    return fail(h, FDVLM_ERR_STATE, "%d masked positions left after %d steps (a masked position 0 under pred_shift = 1 cannot be revealed)",
                h->n_remaining, h->info_host[5]);
  return FDVLM_OK;
}

static int commit_step_core(fdvlm_t* h, int Bn, const int32_t* init_dev, const fdvlm_step_params* p, int want_logits);

extern "C" int fdvlm_commit_decode_block(fdvlm_t* h, int block_size, const int32_t* init_tokens, const fdvlm_step_params* p,
                                         int32_t* block_tokens, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!h->block_open) return fdvlm_decode_block(h, block_size, init_tokens, p, block_tokens, info);
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "commit_decode_block needs the host info struct");
  int rc = check_step_params(h, p);
  if (rc) return rc;
  if (!h->use_graphs) return fail(h, FDVLM_ERR_UNSUPPORTED, "decode_block needs the tensor-core path on a non-default stream");
  rc = commit_step_core(h, block_size, init_tokens, p, 0);      // the finished block's commit + this block's first step
  if (rc) return rc;
  rc = sync_info(h);                                            // what the first step left masked decides whether the loop runs
  if (rc) return rc;
  return decode_loop_rest(h, block_size, p, block_tokens, info, 1);
}

extern "C" int fdvlm_block_step_host(fdvlm_t* h, const fdvlm_step_params* p, float* conf_host, int32_t* pred_host,
                                     uint8_t* unmask_host, int32_t* block_tokens_host, fdvlm_step_info* info) {
  int rc = step_core(h, p, 0);
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

// Causal pass over the finished block with cache update.  all_rows: confidence / prediction of every row are left in
// h->conf / h->pred (and, with want_logits, all rows' logits in h->logits); else only the last row's logits.
static int commit_core(fdvlm_t* h, int all_rows, int want_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "commit without an open block");
  if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "commit with %d masked positions left", h->n_remaining);
  const int B = h->block_size;
  h->launches = 0;
  int rc = stage_rows(h, 0, B, h->blk_tokens, nullptr);
  if (rc) return rc;
  rc = forward_rows(h, B, MODE_CAUSAL, all_rows ? B : (want_logits ? 1 : 0), all_rows ? want_logits : 1);
  if (rc) return rc;
  h->cache_len += B;
  h->block_open = 0;
  h->block_size = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_commit_block(fdvlm_t* h, float* next_logits) {
  int rc = commit_core(h, 0, next_logits != nullptr);
  if (rc) return rc;
  if (next_logits) CU(h, cudaMemcpyAsync(next_logits, h->logits, (size_t)h->cfg.vocab * 4, cudaMemcpyDeviceToDevice, h->st));
  return FDVLM_OK;
}

extern "C" int fdvlm_commit_block_verify(fdvlm_t* h, int32_t* row_pred, float* row_conf, float* next_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  const int B = h->block_size;
  int rc = commit_core(h, 1, next_logits != nullptr);
  if (rc) return rc;
  const cudaMemcpyKind DD = cudaMemcpyDeviceToDevice;
  if (row_pred) CU(h, cudaMemcpyAsync(row_pred, h->pred, (size_t)B * 4, DD, h->st));
  if (row_conf) CU(h, cudaMemcpyAsync(row_conf, h->conf, (size_t)B * 4, DD, h->st));
  if (next_logits) CU(h, cudaMemcpyAsync(next_logits, h->logits + (size_t)(B - 1) * h->cfg.vocab, (size_t)h->cfg.vocab * 4, DD, h->st));
  return FDVLM_OK;
}

// ---- commit of the finished block + first denoise step of the next block as ONE forward ---------------------------------
// Rows [finished block ; next block]: the finished rows run causally among themselves and their K / V are staged at the
// positions they are committed to; the next block's rows read them, the cache and one another.  Every weight byte is
// streamed once instead of twice.
static int commit_step_core(fdvlm_t* h, int Bn, const int32_t* init_dev, const fdvlm_step_params* p, int want_logits) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  int prc = check_step_params(h, p);
  if (prc) return prc;
  if (!h->block_open) return fail(h, FDVLM_ERR_STATE, "commit without an open block");
  if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "commit with %d masked positions left", h->n_remaining);
  const int Bc = h->block_size, n = Bc + Bn;
  if (Bn < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "block_size must be positive");
  if (n > h->cfg.max_block || n > 64)
    return fail(h, FDVLM_ERR_CAPACITY, "commit + step in one forward needs %d + %d rows; max_block is %d (and at most 64)", Bc, Bn,
                h->cfg.max_block);
  if (h->cache_len + n > h->cfg.max_seq)
    return fail(h, FDVLM_ERR_CAPACITY, "block: %d + %d exceed max_seq %d", h->cache_len, n, h->cfg.max_seq);
  h->launches = 0;
  launch_fuse_begin(h->blk_tokens, h->blk_masked, Bc, init_dev, Bn, h->cfg.mask_id, h->f_rows, h->f_mask, h->info, h->st);
  CU(h, cudaGetLastError());
  if (init_dev) {                  // the masked count of the given tokens
    int rc = sync_info(h);
    if (rc) return rc;
  } else {
    h->n_remaining = Bn;
  }
  int rc = stage_rows(h, 0, n, h->f_rows, nullptr);
  if (rc) return rc;
  rc = forward_rows(h, n, MODE_FUSED, n, want_logits);
  if (rc) return rc;
  launch_select(h->conf + Bc, h->pred + Bc, h->blk_tokens, h->blk_masked, h->unmask, h->info, Bn, (int)p->rule, p->threshold, p->k,
                h->st, p->pred_shift);
  h->launches += 2;
  CU(h, cudaGetLastError());
  h->cache_len += Bc;
  h->block_size = Bn;
  h->block_open = 1;
  h->step_index = 1;
  return FDVLM_OK;
}

extern "C" int fdvlm_commit_begin_step(fdvlm_t* h, float* next_logits, int next_block_size, const int32_t* next_init_tokens,
                                       const fdvlm_step_params* p, float* logits, float* conf, int32_t* pred, uint8_t* unmask,
                                       int32_t* block_tokens, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  const int Bc = h->block_size, B = next_block_size;
  int rc = commit_step_core(h, B, next_init_tokens, p, (logits != nullptr || next_logits != nullptr) ? 1 : 0);
  if (rc) return rc;
  const size_t V = (size_t)h->cfg.vocab;
  const cudaMemcpyKind DD = cudaMemcpyDeviceToDevice;
  if (next_logits) CU(h, cudaMemcpyAsync(next_logits, h->logits + (size_t)(Bc - 1) * V, V * 4, DD, h->st));
  if (logits) CU(h, cudaMemcpyAsync(logits, h->logits + (size_t)Bc * V, (size_t)B * V * 4, DD, h->st));
  if (conf) CU(h, cudaMemcpyAsync(conf, h->conf + Bc, (size_t)B * 4, DD, h->st));
  if (pred) CU(h, cudaMemcpyAsync(pred, h->pred + Bc, (size_t)B * 4, DD, h->st));
  if (unmask) CU(h, cudaMemcpyAsync(unmask, h->unmask, (size_t)B, DD, h->st));
  if (block_tokens) CU(h, cudaMemcpyAsync(block_tokens, h->blk_tokens, (size_t)B * 4, DD, h->st));
  return finish_info(h, info);
}

extern "C" int fdvlm_commit_begin_step_host(fdvlm_t* h, int next_block_size, const int32_t* next_init_tokens_host,
                                            const fdvlm_step_params* p, float* conf_host, int32_t* pred_host,
                                            uint8_t* unmask_host, int32_t* block_tokens_host, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  const int Bc = h->block_size, B = next_block_size;
  if (B < 1 || B > 64) return fail(h, FDVLM_ERR_INVALID_ARG, "block_size out of range");
  const int32_t* init_dev = nullptr;
  if (next_init_tokens_host) {
    memcpy(h->host_stage, next_init_tokens_host, (size_t)B * 4);
    CU(h, cudaMemcpyAsync(h->init_stage, h->host_stage, (size_t)B * 4, cudaMemcpyHostToDevice, h->st));
    init_dev = h->init_stage;
  }
  int rc = commit_step_core(h, B, init_dev, p, 0);
  if (rc) return rc;
  char* s = h->host_stage;  // [conf 256 | pred 256 | tokens 256 | unmask 64]
  const cudaMemcpyKind DH = cudaMemcpyDeviceToHost;
  if (conf_host) CU(h, cudaMemcpyAsync(s, h->conf + Bc, (size_t)B * 4, DH, h->st));
  if (pred_host) CU(h, cudaMemcpyAsync(s + 256, h->pred + Bc, (size_t)B * 4, DH, h->st));
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

extern "C" int fdvlm_commit_decode_block_topk(fdvlm_t* h, int block_size, const int32_t* init_tokens, int k, int pred_shift,
                                              int32_t* block_tokens, fdvlm_step_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!h->block_open) return fdvlm_decode_block_topk(h, block_size, init_tokens, k, pred_shift, block_tokens, info);
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "commit_decode_block_topk needs the host info struct");
  if (k < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "top-k needs k >= 1");
  fdvlm_step_params p;
  p.rule = FDVLM_RULE_TOPK; p.threshold = 0.f; p.k = k; p.pred_shift = pred_shift;
  int rc = commit_step_core(h, block_size, init_tokens, &p, 0);
  if (rc) return rc;
  const int steps = (h->n_remaining + k - 1) / k;      // of which the first has just run
  int launches = h->launches;
  for (int s = 1; s < steps; ++s) {
    h->n_remaining = 1;            // the device keeps the true count; the host checks it once, below
    rc = step_core(h, &p, 0);
    if (rc) return rc;
    launches += h->launches;
  }
  h->launches = launches;
  if (block_tokens) CU(h, cudaMemcpyAsync(block_tokens, h->blk_tokens, (size_t)block_size * 4, cudaMemcpyDeviceToDevice, h->st));
  rc = sync_info(h);
  if (rc) return rc;
  info->n_unmasked = h->info_host[0]; info->n_remaining = h->info_host[1]; info->step_index = h->info_host[2];
  if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "%d masked positions left after %d top-%d steps", h->n_remaining, steps, k);
  return FDVLM_OK;
}

extern "C" int fdvlm_truncate(fdvlm_t* h, int new_len) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (h->block_open) return fail(h, FDVLM_ERR_STATE, "truncate inside an open block");
  if (new_len < 0 || new_len > h->cache_len) return fail(h, FDVLM_ERR_INVALID_ARG, "truncate to %d of %d committed positions", new_len, h->cache_len);
  h->cache_len = new_len;
  return FDVLM_OK;
}

extern "C" int fdvlm_spec_block(fdvlm_t* h, int block_size, int32_t seed_token, int32_t* draft_tokens, int32_t* verify_pred,
                                fdvlm_spec_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "spec_block needs the host info struct");
  if (seed_token < 0 || seed_token >= h->cfg.vocab || seed_token == h->cfg.mask_id)
    return fail(h, FDVLM_ERR_INVALID_ARG, "seed token %d is not a vocabulary token", (int)seed_token);
  int rc = block_begin_common(h, block_size);
  if (rc) return rc;
  const int B = block_size, L0 = h->cache_len;
  int32_t init[64];
  init[0] = seed_token;
  for (int i = 1; i < B; ++i) init[i] = h->cfg.mask_id;
  rc = fdvlm_block_begin_host(h, B, init);
  if (rc) return rc;
  if (B > 1) {
    // draft: one denoise pass, shift-by-one, every masked position filled (threshold below any confidence)
    fdvlm_step_params p;
    p.rule = FDVLM_RULE_THRESHOLD; p.threshold = -1.f; p.k = 0; p.pred_shift = 1;
    rc = step_core(h, &p, 0);
    if (rc) return rc;
    rc = sync_info(h);
    if (rc) return rc;
    if (h->n_remaining != 0) return fail(h, FDVLM_ERR_STATE, "draft pass left %d masked positions", h->n_remaining);
  }
  const cudaMemcpyKind DD = cudaMemcpyDeviceToDevice;
  if (draft_tokens) CU(h, cudaMemcpyAsync(draft_tokens, h->blk_tokens, (size_t)B * 4, DD, h->st));
  // verify: causal pass with cache update, predictions of every row
  const int draft_launches = h->launches;
  rc = commit_core(h, 1, 0);
  if (rc) return rc;
  if (verify_pred) CU(h, cudaMemcpyAsync(verify_pred, h->pred, (size_t)B * 4, DD, h->st));
  launch_accept(h->pred, h->blk_tokens, B, h->init_stage, h->st);
  h->launches += draft_launches + 1;
  CU(h, cudaGetLastError());
  CU(h, cudaMemcpyAsync(h->host_stage, h->init_stage, 8, cudaMemcpyDeviceToHost, h->st));
  rc = sync_info(h);              // synchronises, and reports a timed-out device wait of either pass
  if (rc) return rc;
  const int k = ((const int32_t*)h->host_stage)[0];
  if (k < 1 || k > B) return fail(h, FDVLM_ERR_CUDA, "accept kernel returned %d", k);
  h->cache_len = L0 + k;          // crop: the rows after the accepted prefix are dropped
  info->accepted = k;
  info->next_token = ((const int32_t*)h->host_stage)[1];
  info->cache_len = h->cache_len;
  return FDVLM_OK;
}

// ---- quadratic self-speculative decoding (Appendix B, Alg. 2) --------------------------------------------------------
extern "C" int fdvlm_quad_begin(fdvlm_t* h, int block_size, int32_t first_token, int chain, int32_t* draft) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  const int B = block_size;
  if (B < 1) return fail(h, FDVLM_ERR_INVALID_ARG, "block_size must be positive");
  if (first_token < 0 || first_token >= h->cfg.vocab || first_token == h->cfg.mask_id)
    return fail(h, FDVLM_ERR_INVALID_ARG, "first token %d is not a vocabulary token", (int)first_token);
  if (B * (B + 1) > h->cfg.max_block || B * (B + 1) > 64)
    return fail(h, FDVLM_ERR_CAPACITY, "quadratic decoding runs B (B + 1) = %d rows per forward; max_block is %d (and at most 64)",
                B * (B + 1), h->cfg.max_block);
  if (h->block_open) return fail(h, FDVLM_ERR_STATE, "a block is open");
  if (h->cache_len + B * (B + 1) > h->cfg.max_seq)
    return fail(h, FDVLM_ERR_CAPACITY, "quad: %d + %d exceed max_seq %d", h->cache_len, B * (B + 1), h->cfg.max_seq);
  // step 1: B mask tokens after the prompt, one denoise pass; the cache keeps the prompt only
  h->launches = 0;
  launch_init_block(h->blk_tokens, h->blk_masked, h->info, nullptr, B, h->cfg.mask_id, 0, h->st);
  int rc = stage_rows(h, 0, B, h->blk_tokens, nullptr);
  if (rc) return rc;
  rc = forward_rows(h, B, MODE_BIDIR, B, 0);
  if (rc) return rc;
  launch_quad_first_draft(h->pred, first_token, B, h->q_d, h->st);
  launch_quad_layout(B, chain ? 1 : 0, h->q_mask, h->q_pos_off, h->st);
  h->launches += 3;
  CU(h, cudaGetLastError());
  if (draft) CU(h, cudaMemcpyAsync(draft, h->q_d, (size_t)B * 4, cudaMemcpyDeviceToDevice, h->st));
  rc = sync_info(h);
  if (rc) return rc;
  h->quad_B = B;
  return FDVLM_OK;
}

extern "C" int fdvlm_quad_set_draft(fdvlm_t* h, const int32_t* draft) {
  if (!h || !draft) return FDVLM_ERR_INVALID_ARG;
  if (!h->quad_B) return fail(h, FDVLM_ERR_STATE, "no quadratic decode is open");
  CU(h, cudaMemcpyAsync(h->q_d, draft, (size_t)h->quad_B * 4, cudaMemcpyDeviceToDevice, h->st));
  return FDVLM_OK;
}

extern "C" int fdvlm_quad_step(fdvlm_t* h, int32_t* accepted_tokens, int32_t* next_draft, int32_t* row_pred, float* logits,
                               fdvlm_quad_info* info) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (!info) return fail(h, FDVLM_ERR_INVALID_ARG, "quad_step needs the host info struct");
  if (!h->quad_B) return fail(h, FDVLM_ERR_STATE, "no quadratic decode is open");
  if (h->block_open) return fail(h, FDVLM_ERR_STATE, "a block is open");
  const int B = h->quad_B, n = B * (B + 1), L0 = h->cache_len;
  if (L0 + n > h->cfg.max_seq) return fail(h, FDVLM_ERR_CAPACITY, "quad: %d + %d exceed max_seq %d", L0, n, h->cfg.max_seq);
  h->launches = 0;
  launch_quad_build(h->q_d, B, h->cfg.mask_id, h->blk_tokens, h->blk_masked, h->st);
  int rc = stage_rows(h, 0, n, h->blk_tokens, nullptr);
  if (rc) return rc;
  rc = forward_rows(h, n, MODE_MASKED, n, logits != nullptr);
  if (rc) return rc;
  const cudaMemcpyKind DD = cudaMemcpyDeviceToDevice;
  if (logits) CU(h, cudaMemcpyAsync(logits, h->logits, (size_t)n * h->cfg.vocab * 4, DD, h->st));
  if (row_pred) CU(h, cudaMemcpyAsync(row_pred, h->pred, (size_t)n * 4, DD, h->st));
  // verify loop on the device; the accepted tokens land in init_stage[8 ..], the count in init_stage[0]
  launch_quad_accept(h->pred, h->q_d, B, h->init_stage + 8, h->init_stage, h->st);
  h->launches += 2;
  CU(h, cudaGetLastError());
  if (accepted_tokens) CU(h, cudaMemcpyAsync(accepted_tokens, h->init_stage + 8, (size_t)B * 4, DD, h->st));
  if (next_draft) CU(h, cudaMemcpyAsync(next_draft, h->q_d, (size_t)B * 4, DD, h->st));
  CU(h, cudaMemcpyAsync(h->host_stage, h->init_stage, 4, cudaMemcpyDeviceToHost, h->st));
  rc = sync_info(h);              // synchronises, and reports a timed-out device wait
  if (rc) return rc;
  const int k = ((const int32_t*)h->host_stage)[0];
  if (k < 1 || k > B) return fail(h, FDVLM_ERR_CUDA, "verify kernel returned %d", k);
  // the first tokens are the first rows of the forward: the K / V of d_0 .. d_{k-1} already sit at cache rows L0 .. L0+k-1
  h->cache_len = L0 + k;
  info->accepted = k;
  info->cache_len = h->cache_len;
  return FDVLM_OK;
}

extern "C" int fdvlm_quad_end(fdvlm_t* h) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  h->quad_B = 0;
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
extern "C" int fdvlm_profile_enable(fdvlm_t* h, int mode) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  if (mode < 0 || mode > 2) return fail(h, FDVLM_ERR_INVALID_ARG, "profile mode is 0, 1 or 2");
  if (mode == 2 && !h->use_tc) return fail(h, FDVLM_ERR_UNSUPPORTED, "in-chain timing covers the tensor-core path only");
  h->prof_on = mode;
  h->prof_used = 0;
  h->stamp_used = 0;
  return FDVLM_OK;
}

extern "C" int fdvlm_profile_read_chain(fdvlm_t* h, fdvlm_kernel_record* records, int cap, int* n) {
  if (!h) return FDVLM_ERR_INVALID_ARG;
  CU(h, cudaStreamSynchronize(h->st));
  const int used = h->stamp_used;
  if (n) *n = used;
  if (!records || cap <= 0 || used == 0) return FDVLM_OK;
  std::vector<KStamp> host((size_t)used);
  CU(h, cudaMemcpy(host.data(), h->stamps, sizeof(KStamp) * used, cudaMemcpyDeviceToHost));
  unsigned long long t0 = ~0ull;
  for (const KStamp& k : host) if (k.start < t0) t0 = k.start;
  for (int i = 0; i < used && i < cap; ++i) {
    const KStamp& k = host[i];
    records[i].kind = h->stamp_kind[i];
    records[i].start_us = (k.start == ~0ull) ? -1.0 : (double)(k.start - t0) * 1e-3;
    records[i].released_us = (k.released == ~0ull) ? -1.0 : (double)(k.released - t0) * 1e-3;
    records[i].end_us = (k.end_inv == ~0ull) ? -1.0 : (double)(~k.end_inv - t0) * 1e-3;
  }
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

// ---- measurement yardstick ------------------------------------------------------------------------------
extern "C" int fdvlm_util_stream_read(const void* device_buf, size_t bytes, void* device_sink, void* cuda_stream) {
  if (!device_buf || !device_sink || bytes < 16 || ((uintptr_t)device_buf & 15)) return FDVLM_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return FDVLM_ERR_CUDA;
  launch_stream_read(device_buf, bytes, (unsigned*)device_sink, sms * 8, (cudaStream_t)cuda_stream);
  return cudaGetLastError() == cudaSuccess ? FDVLM_OK : FDVLM_ERR_CUDA;
}

// ---- single operators ---------------------------------------------------------------------------------
extern "C" size_t fdvlm_op_linear_workspace_bytes(int m, int n, int k, fdvlm_dtype dtype) {
  if (m < 1 || n < 1 || k < 1) return 0;
  return linear_workspace_bytes(m, n, k, (int)dtype);
}

extern "C" int fdvlm_op_linear(const void* x, const void* w, const float* scale, const float* bias, float* y, int m,
                               int n, int k, fdvlm_dtype dtype, void* workspace, void* cuda_stream) {
  if (!x || !w || !y || m < 1 || m > 64 || n < 1 || k < 8 || (k % 8)) return FDVLM_ERR_INVALID_ARG;
  if (dtype != FDVLM_F32 && dtype != FDVLM_BF16 && dtype != FDVLM_W_FP8E4M3 && dtype != FDVLM_W8A8_FP8E4M3) return FDVLM_ERR_INVALID_ARG;
  if ((dtype == FDVLM_W_FP8E4M3 || dtype == FDVLM_W8A8_FP8E4M3) && !scale) return FDVLM_ERR_INVALID_ARG;
  LinearArgs a;
  a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = n; a.k = k; a.ldy = n; a.accumulate = 0;
  a.dtype = (int)dtype; a.workspace = workspace; a.workspace_bytes = linear_workspace_bytes(m, n, k, (int)dtype);
  if (!workspace) return FDVLM_ERR_INVALID_ARG;
  cudaError_t e;
  int r = launch_linear(a, (cudaStream_t)cuda_stream, &e);
  if (r < 0) return e == cudaErrorNotSupported ? FDVLM_ERR_UNSUPPORTED : FDVLM_ERR_CUDA;
  return FDVLM_OK;
}

extern "C" size_t fdvlm_op_attention_workspace_bytes(int n_rows, int n_q_heads, int n_kv_heads, int head_dim) {
  if (n_rows < 1 || n_q_heads < 1 || n_kv_heads < 1 || (n_q_heads % n_kv_heads)) return 0;
  return attention_workspace_bytes(n_rows, n_q_heads, n_kv_heads, head_dim);
}

extern "C" int fdvlm_op_attention(const void* q, const void* k_cache, const void* v_cache, void* out, int n_rows,
                                  int cache_len, int max_seq, int n_q_heads, int n_kv_heads, int head_dim, int causal,
                                  fdvlm_dtype dtype, fdvlm_kv_dtype kv_dtype, void* workspace, void* cuda_stream) {
  if (!q || !k_cache || !v_cache || !out || n_rows < 1 || n_rows > 64 || cache_len < 0 || cache_len + n_rows > max_seq ||
      n_q_heads < 1 || n_kv_heads < 1 || (n_q_heads % n_kv_heads) || (head_dim != 64 && head_dim != 128))
    return FDVLM_ERR_INVALID_ARG;
  if (dtype != FDVLM_F32 && dtype != FDVLM_BF16 && dtype != FDVLM_W_FP8E4M3) return FDVLM_ERR_INVALID_ARG;
  if (kv_dtype != FDVLM_KV_BF16 && kv_dtype != FDVLM_KV_F16) return FDVLM_ERR_INVALID_ARG;
  AttnArgs a;
  memset(&a, 0, sizeof(a));
  a.kv_type = (int)kv_dtype; a.out_fmt = kv_dtype == FDVLM_KV_F16 ? XF_F16 : XF_BF16; a.long_cache = -1;
  a.q = q; a.kc = k_cache; a.vc = v_cache; a.out = out; a.n = n_rows; a.cache_len = cache_len; a.max_seq = max_seq;
  a.hq = n_q_heads; a.hkv = n_kv_heads; a.d = head_dim; a.causal = causal ? 1 : 0; a.dtype = (int)dtype; a.workspace = workspace;
  cudaError_t e;
  int r = launch_attention(a, (cudaStream_t)cuda_stream, &e);
  return r < 0 ? FDVLM_ERR_CUDA : FDVLM_OK;
}
