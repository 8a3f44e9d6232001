// Split-KV, block-masked GQA attention for the bf16 path.
//
// One CTA = (KV head, group of query heads that share it, chunk of keys).  The CTA's rows are the
// block's n rows of each of its query heads (<= 64 rows in all): K/V of the chunk are staged once in
// shared memory (16-byte cp.async, XOR-swizzled rows, double buffered) and reused by every row.
// Scores and P.V run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with an online softmax in fp32;
// each CTA leaves an unnormalised partial (O, running max, running sum) and a small second kernel
// merges the chunks.  The in-block mask is applied by key index: denoise rows see all L + n keys,
// commit / prefill rows see keys <= L + i.
#include "attn_core.cuh"
#include "kernels.h"

namespace fdk {

// len_ptr (nullable): the cache length is read from device memory instead of L, and the chunking is derived from
// it and `bound` (= gridDim.x) on the device -- lets one captured launch serve every cache length.
template <int D, typename T>
__global__ void __launch_bounds__(128) attn_mma_kernel(const T* __restrict__ q, const T* __restrict__ kc,
                                                       const T* __restrict__ vc, float* __restrict__ part_o,
                                                       float2* __restrict__ part_ml, int n, int L, int max_seq, int hq,
                                                       int hkv, int qh, int chunk_keys, int n_chunks, int causal,
                                                       const int* __restrict__ len_ptr, KStamp* stamp) {
  extern __shared__ __align__(128) uint8_t smem[];
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  if (len_ptr) {   // the length word is written before the forward starts, not by a predecessor kernel
    L = *len_ptr;
    attn_chunking(L + n, (int)gridDim.x, &chunk_keys, &n_chunks);
  }
  if ((int)blockIdx.x >= n_chunks) { pdl_wait(); return; }
  attn_item<D, T, true>(q, kc, vc, part_o, part_ml, n, L, max_seq, hq, hkv, qh, chunk_keys, n_chunks, causal, blockIdx.x, blockIdx.y,
                        blockIdx.z, (uint32_t)__cvta_generic_to_shared(smem), threadIdx.x);
  if (threadIdx.x == 0) stamp_end(stamp);
}

// out[i][head] = sum_c w_c O_c / sum_c w_c l_c, w_c = 2^(m_c - max_c m_c): one warp per (row, head), four per CTA
template <int D>
__global__ void __launch_bounds__(128) attn_combine_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml,
                                                          void* __restrict__ out, size_t lo_off, int fmt, int n, int hq, int n_chunks,
                                                          const int* __restrict__ len_ptr, int bound, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  if (len_ptr) {
    int ck;
    attn_chunking(*len_ptr + n, bound, &ck, &n_chunks);
  }
  pdl_wait();
  if (threadIdx.x == 0) stamp_released(stamp);
  const int p = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (p < n * hq) {
    const int i = p / hq, head = p % hq;
    attn_merge_warp<D>(part_o, part_ml, out, ((size_t)i * hq + head) * D, lo_off, fmt, ((size_t)head * n + i) * n_chunks, n_chunks,
                       threadIdx.x & 31);
  }
  __syncthreads();
  if (threadIdx.x == 0) stamp_end(stamp, true);
}

// ---- host side -------------------------------------------------------------------------------------
struct AttnPlan { int qh, groups, chunk_keys, n_chunks, bound; };

static int attn_max_chunks(int n, int hq, int hkv) {
  const int G = hq / hkv;
  int qh = 1;
  for (int c = G; c >= 1; --c)
    if (c * n <= AT_ROWS) { qh = c; break; }
  return ceil_div(2 * 148, hkv * ceil_div(G, qh));
}

static AttnPlan attn_plan(int n, int T, int hq, int hkv) {
  const int G = hq / hkv;
  AttnPlan p;
  p.qh = 1;
  for (int c = G; c >= 1; --c)                 // most heads per CTA that still fit 64 rows
    if (c * n <= AT_ROWS) { p.qh = c; break; }
  p.groups = ceil_div(G, p.qh);
  p.bound = attn_max_chunks(n, hq, hkv);
  attn_chunking(T, p.bound, &p.chunk_keys, &p.n_chunks);
  return p;
}

size_t attention_mma_workspace_bytes(int n, int hq, int hkv, int d) {
  size_t worst = 0;
  for (int m = 1; m <= n; ++m) {
    size_t slots = (size_t)hq * m * attn_max_chunks(m, hq, hkv);
    if (slots > worst) worst = slots;
  }
  return worst * ((size_t)d * 4 + 8) + 256;
}

template <int D, typename T>
static cudaError_t attn_launch_t(const AttnArgs& a, const AttnPlan& p, cudaStream_t st) {
  // with the length on the device the grid is sized for the most chunks any length can give
  int grid_x = p.n_chunks;
  if (a.len_ptr) { grid_x = p.bound; const int tmax = ceil_div(a.max_seq, AT_KEYS); if (grid_x > tmax) grid_x = tmax; }
  const size_t slots = (size_t)a.hq * a.n * grid_x;
  float* part_o = (float*)a.workspace;
  float2* part_ml = (float2*)((char*)a.workspace + ((slots * D * 4 + 255) / 256) * 256);
  const int smem = AT_ROWS * D * 2 + 4 * AT_KEYS * D * 2;
  static bool attr_set[MAX_DEVICES] = {};
  cudaError_t e = ensure_dynamic_smem(attn_mma_kernel<D, T>, smem, attr_set);
  if (e != cudaSuccess) return e;
  dim3 grid(grid_x, p.groups, a.hkv);
  e = launch_pdl(attn_mma_kernel<D, T>, grid, dim3(128), (size_t)smem, st, (const T*)a.q, (const T*)a.kc, (const T*)a.vc,
                 part_o, part_ml, a.n, a.cache_len, a.max_seq, a.hq, a.hkv, p.qh, p.chunk_keys, p.n_chunks, a.causal, a.len_ptr, a.stamp);
  if (e != cudaSuccess) return e;
  e = launch_pdl(attn_combine_kernel<D>, dim3((a.n * a.hq + 3) / 4), dim3(128), 0, st, (const float*)part_o, (const float2*)part_ml,
                 a.out, a.out_lo_off, a.out_fmt, a.n, a.hq, p.n_chunks, a.len_ptr, grid_x, a.stamp ? a.stamp + 1 : nullptr);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

int launch_attention_mma(const AttnArgs& a, cudaStream_t st, cudaError_t* err) {
  const AttnPlan p = attn_plan(a.n, a.cache_len + a.n, a.hq, a.hkv);
  if (!a.workspace) { *err = cudaErrorInvalidValue; return -1; }
  if (a.kv_type == KV_F16) *err = (a.d == 128) ? attn_launch_t<128, __half>(a, p, st) : attn_launch_t<64, __half>(a, p, st);
  else *err = (a.d == 128) ? attn_launch_t<128, bf16>(a, p, st) : attn_launch_t<64, bf16>(a, p, st);
  return *err == cudaSuccess ? 2 : -1;
}

}  // namespace fdk
