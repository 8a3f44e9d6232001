// CUDA-core (SIMT) kernels of the denoise step: the exact-fp32 path of the fp32 configuration and
// the small fused glue of every configuration (embedding gather, RMSNorm, rotary + KV staging,
// SwiGLU, softmax-max confidence / argmax, unmask selection).
#include "common.cuh"
#include "kernels.h"

namespace fdk {

// ================================================================================================
// small-M linear, CUDA-core version.  Register-tiled: CTA tile BM x 64 outputs, BK = 32 deep.
// Used for fp32 weights (TF32 tensor cores would miss the 1e-4 parity bound of that path) and for
// shapes the tensor-core kernel does not take.
// ================================================================================================
template <typename T> struct Vec8;
template <> struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, float* o) {
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
  }
};
template <> struct Vec8<bf16> {
  static __device__ __forceinline__ void load(const bf16* p, float* o) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const unsigned u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = __uint_as_float(u[i] << 16);
      o[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
  }
};
template <> struct Vec8<fp8e4m3> {
  static __device__ __forceinline__ void load(const fp8e4m3* p, float* o) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    const unsigned u[2] = {v.x, v.y};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      fp8e4m3 e;
      e.b = (uint8_t)((u[i >> 2] >> (8 * (i & 3))) & 0xffu);
      o[i] = to_f32(e);
    }
  }
};

constexpr int SBN = 64, SBK = 32;

template <typename WT, typename XT, int BM>
__global__ void __launch_bounds__((BM / 4) * 16)
linear_simt_kernel(const XT* __restrict__ x, const WT* __restrict__ w, float* __restrict__ part,
                   int m, int N, int K, int k_per_split) {
  constexpr int NT = (BM / 4) * 16;
  __shared__ __align__(16) float xs[SBK][BM + 4];
  __shared__ __align__(16) float ws[SBK][SBN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int n0 = blockIdx.x * SBN;
  const int kb = blockIdx.y * k_per_split;
  const int ke = min(K, kb + k_per_split);
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = kb; k0 < ke; k0 += SBK) {
    // W tile: 64 rows x 32 k as 256 vectors of 8; vector v -> row v % 64, k-quarter v / 64
    for (int v = tid; v < SBN * (SBK / 8); v += NT) {
      int r = v % SBN, kq = v / SBN;
      int n = n0 + r, k = k0 + kq * 8;
      float f[8];
      if (n < N && k < ke) Vec8<WT>::load(w + (size_t)n * K + k, f);
      else {
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) ws[kq * 8 + i][r] = f[i];
    }
    for (int v = tid; v < BM * (SBK / 8); v += NT) {
      int r = v % BM, kq = v / BM;
      int k = k0 + kq * 8;
      float f[8];
      if (r < m && k < ke) Vec8<XT>::load(x + (size_t)r * K + k, f);
      else {
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) xs[kq * 8 + i][r] = f[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SBK; ++kk) {
      float4 xv = *reinterpret_cast<const float4*>(&xs[kk][ty * 4]);
      float4 wv = *reinterpret_cast<const float4*>(&ws[kk][tx * 4]);
      const float xa[4] = {xv.x, xv.y, xv.z, xv.w}, wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xa[i], wa[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* dst = part + (size_t)blockIdx.y * m * N;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int r = ty * 4 + i;
    if (r >= m) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int n = n0 + tx * 4 + j;
      if (n < N) dst[(size_t)r * N + n] = acc[i][j];
    }
  }
}

// y[r, n] = (accumulate ? y : 0) + (sum_s part[s][r][n]) * scale[n] + bias[n]; fixed summation order.
__global__ void splitk_epilogue_kernel(const float* __restrict__ part, int S, int m, int N,
                                       const float* __restrict__ scale, const float* __restrict__ bias,
                                       float* __restrict__ y, int ldy, int accumulate, const float* __restrict__ row_amax) {
  pdl_trigger();
  pdl_wait();
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t total = (size_t)m * N;
  if (idx >= total) return;
  int r = (int)(idx / N), n = (int)(idx % N);
  float s = 0.f;
  for (int i = 0; i < S; ++i) s += part[(size_t)i * total + idx];
  if (scale) s *= scale[n];
  if (row_amax) s *= row_amax[r] > 0.f ? __fdiv_rn(row_amax[r], 448.f) : 1.f;   // sums of e4m3 code products: the row's scale
  if (bias) s += bias[n];
  float* o = y + (size_t)r * ldy + n;
  *o = accumulate ? (*o + s) : s;
}

void launch_splitk_epilogue(const float* part, int S, int m, int n, const float* scale, const float* bias, float* y, int ldy,
                            int accumulate, cudaStream_t st, const float* row_amax) {
  size_t total = (size_t)m * n;
  splitk_epilogue_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(part, S, m, n, scale, bias, y, ldy, accumulate, row_amax);
}

static void simt_plan(int m, int n, int k, int* bm, int* splits, int* kps) {
  *bm = m <= 16 ? 16 : (m <= 32 ? 32 : 64);
  int tiles = ceil_div(n, SBN);
  int kblocks = ceil_div(k, SBK);
  int want = ceil_div(2 * 148, tiles);                 // at least ~2 CTAs per SM when K allows
  int s = want < 1 ? 1 : want;
  int max_s = kblocks / 8 > 0 ? kblocks / 8 : 1;       // >= 256 deep per split
  if (s > max_s) s = max_s;
  if (s > 16) s = 16;
  int per = ceil_div(kblocks, s) * SBK;
  *kps = per;
  *splits = ceil_div(k, per);
}

size_t simt_workspace_bytes(int m, int n, int k) {
  int bm, s, kps;
  simt_plan(m, n, k, &bm, &s, &kps);
  return (size_t)s * m * n * sizeof(float);
}

template <typename WT, typename XT>
static void simt_dispatch(const LinearArgs& a, int bm, dim3 grid, float* part, int kps, cudaStream_t st) {
  const XT* x = (const XT*)a.x;
  const WT* w = (const WT*)a.w;
  if (bm == 16) linear_simt_kernel<WT, XT, 16><<<grid, 64, 0, st>>>(x, w, part, a.m, a.n, a.k, kps);
  else if (bm == 32) linear_simt_kernel<WT, XT, 32><<<grid, 128, 0, st>>>(x, w, part, a.m, a.n, a.k, kps);
  else linear_simt_kernel<WT, XT, 64><<<grid, 256, 0, st>>>(x, w, part, a.m, a.n, a.k, kps);
}

int launch_linear_simt(const LinearArgs& a, cudaStream_t st, cudaError_t* err) {
  int bm, s, kps;
  simt_plan(a.m, a.n, a.k, &bm, &s, &kps);
  size_t need = (size_t)s * a.m * a.n * sizeof(float);
  if (need > a.workspace_bytes || a.workspace == nullptr) { *err = cudaErrorInvalidValue; return -1; }
  float* part = (float*)a.workspace;
  dim3 grid(ceil_div(a.n, SBN), s);
  if (a.dtype == DT_F32) simt_dispatch<float, float>(a, bm, grid, part, kps, st);
  else if (a.dtype == DT_BF16) simt_dispatch<bf16, bf16>(a, bm, grid, part, kps, st);
  else simt_dispatch<fp8e4m3, bf16>(a, bm, grid, part, kps, st);
  size_t total = (size_t)a.m * a.n;
  splitk_epilogue_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(part, s, a.m, a.n, a.scale, a.bias, a.y,
                                                                         a.ldy, a.accumulate, nullptr);
  *err = cudaGetLastError();
  return *err == cudaSuccess ? 2 : -1;
}

// ================================================================================================
// embedding gather / row conversion
// ================================================================================================
// A token id outside [0, vocab) is not dereferenced: row 0 is read instead and ST_BAD_TOKEN is left in the status word.
__device__ __forceinline__ int checked_token(const int32_t* tokens, int r, int vocab, int* status) {
  const int t = tokens[r];
  if (t >= 0 && t < vocab) return t;
  if (threadIdx.x == 0 && status) atomicCAS(status, 0, ST_BAD_TOKEN);
  return 0;
}
template <typename ET>
__global__ void embed_kernel(const ET* __restrict__ table, const int32_t* __restrict__ tokens,
                             float* __restrict__ h, int hidden, int vocab, int* status) {
  int r = blockIdx.x;
  const ET* src = table + (size_t)(tokens ? checked_token(tokens, r, vocab, status) : r) * hidden;
  for (int c = threadIdx.x; c < hidden; c += blockDim.x) h[(size_t)r * hidden + c] = to_f32(src[c]);
}
void launch_embed(const void* table, const int32_t* tokens, float* h, int n, int hidden, int dtype, int vocab, int* status,
                  cudaStream_t st) {
  if (dtype == DT_F32) embed_kernel<float><<<n, 256, 0, st>>>((const float*)table, tokens, h, hidden, vocab, status);
  else embed_kernel<bf16><<<n, 256, 0, st>>>((const bf16*)table, tokens, h, hidden, vocab, status);
}
void launch_rows_to_f32(const void* rows, float* h, int n, int hidden, int dtype, cudaStream_t st) {
  launch_embed(rows, nullptr, h, n, hidden, dtype, 0, nullptr, st);
}

// ================================================================================================
// RMSNorm: out = x * rsqrt(mean(x^2) + eps) * g, fp32 math, output in the activation type
// ================================================================================================
template <typename AT>
__global__ void rmsnorm_kernel(const float* __restrict__ h, const float* __restrict__ g, AT* __restrict__ out,
                               int hidden, float eps) {
  __shared__ float red[32];
  const float* x = h + (size_t)blockIdx.x * hidden;
  float ss = 0.f;
  for (int c = threadIdx.x; c < hidden; c += blockDim.x) { float v = x[c]; ss = fmaf(v, v, ss); }
  ss = block_sum(ss, red);
  float r = rsqrtf(ss / (float)hidden + eps);
  AT* o = out + (size_t)blockIdx.x * hidden;
  for (int c = threadIdx.x; c < hidden; c += blockDim.x) o[c] = from_f32<AT>(x[c] * r * g[c]);
}
void launch_rmsnorm(const float* h, const float* g, void* out, int n, int hidden, float eps, int dtype, cudaStream_t st) {
  if (dtype == DT_F32) rmsnorm_kernel<float><<<n, 256, 0, st>>>(h, g, (float*)out, hidden, eps);
  else rmsnorm_kernel<bf16><<<n, 256, 0, st>>>(h, g, (bf16*)out, hidden, eps);
}

// ================================================================================================
// rotary table: cs[r][j] = (cos, sin)(pos * theta^(-2j/d)), angles formed in fp64
// ================================================================================================
__global__ void set_len_kernel(int* len_ptr, int value) {
  pdl_trigger();
  pdl_wait();
  *len_ptr = value;
}
void launch_set_len(int* len_ptr, int value, cudaStream_t st) { set_len_kernel<<<1, 1, 0, st>>>(len_ptr, value); }

// cs[r][j] = (cos, sin) of position(r) * theta^(-j / half); position(r) = pos0 + r, or pos0 + pos_off[r] when the rows
// carry their own position ids (Appendix B, Alg. 2: group i of the quadratic input covers positions s+i .. s+i+B)
__global__ void rope_table_kernel(float2* __restrict__ cs, int n, int pos0, int half, double theta, const int* __restrict__ len_ptr,
                                  const int* __restrict__ pos_off, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) { stamp_released(stamp); stamp_end(stamp); }
  if (len_ptr) pos0 = *len_ptr;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n * half) return;
  int r = idx / half, j = idx % half;
  double inv = pow(theta, -(double)j / (double)half);
  double ang = (double)(pos0 + (pos_off ? pos_off[r] : r)) * inv, s, c;
  sincos(ang, &s, &c);
  cs[idx] = make_float2((float)c, (float)s);
}
void launch_rope_table(float* cs, int n, int pos0, int head_dim, float theta, cudaStream_t st, const int* len_ptr, KStamp* stamp,
                       const int* pos_off) {
  int half = head_dim / 2, total = n * half;
  launch_pdl(rope_table_kernel, dim3((total + 127) / 128), dim3(128), 0, st, (float2*)cs, n, pos0, half, (double)theta, len_ptr, pos_off,
             stamp);
}

// rotate-half pairing (j, j + d/2); q -> q buffer, k -> cache K plane, v -> cache V plane
template <typename AT>
__global__ void qkv_post_kernel(const float* __restrict__ qkv, const float2* __restrict__ cs, AT* __restrict__ q,
                                AT* __restrict__ kc, AT* __restrict__ vc, int pos0, int hq, int hkv, int d, int max_seq) {
  int r = blockIdx.x, half = d >> 1;
  int width = (hq + 2 * hkv) * d;
  const float* row = qkv + (size_t)r * width;
  int pairs = (hq + hkv) * half;
  for (int t = threadIdx.x; t < pairs; t += blockDim.x) {
    int head = t / half, j = t % half;
    float2 c = cs[r * half + j];
    float a = row[head * d + j], b = row[head * d + j + half];
    float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
    if (head < hq) {
      AT* o = q + ((size_t)r * hq + head) * d;
      o[j] = from_f32<AT>(ra); o[j + half] = from_f32<AT>(rb);
    } else {
      AT* o = kc + ((size_t)(head - hq) * max_seq + pos0 + r) * d;
      o[j] = from_f32<AT>(ra); o[j + half] = from_f32<AT>(rb);
    }
  }
  const float* vrow = row + (hq + hkv) * d;
  for (int t = threadIdx.x; t < hkv * d; t += blockDim.x) {
    int head = t / d, j = t % d;
    vc[((size_t)head * max_seq + pos0 + r) * d + j] = from_f32<AT>(vrow[t]);
  }
}
void launch_qkv_post(const float* qkv, const float* cs, void* q, void* kc, void* vc, int n, int pos0, int hq, int hkv,
                     int d, int max_seq, int dtype, cudaStream_t st) {
  if (dtype == DT_F32)
    qkv_post_kernel<float><<<n, 256, 0, st>>>(qkv, (const float2*)cs, (float*)q, (float*)kc, (float*)vc, pos0, hq, hkv, d, max_seq);
  else
    qkv_post_kernel<bf16><<<n, 256, 0, st>>>(qkv, (const float2*)cs, (bf16*)q, (bf16*)kc, (bf16*)vc, pos0, hq, hkv, d, max_seq);
}

// ================================================================================================
// Glue of the tensor-core path.  RMSNorm is folded into its consumer GEMM: producers leave xg = h * gain as a GEMM
// input (XF_* storage: bf16 hi + lo planes, or f16) and per-128-column partial sums of h^2 (ssq[row][nt]); the
// consumer's epilogue multiplies by rsqrt(sum(ssq) / hidden + eps).  All sums run in a fixed order => deterministic.
// ================================================================================================
// W8A8 (Sec. 3.4 "System integration"): a projection input row is quantised to e4m3 with the scale max|row| / 448, the
// maximum taken over the values as stored (f16).  Producers leave partial maxima; consumers of code-product sums
// multiply by the scale.
__device__ __forceinline__ float abs_as_f16(float v) { return fabsf(__half2float(__ushort_as_half(f16_bits_sat(v)))); }
__device__ __forceinline__ float scale_of_amax(float amax) { return amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f; }

__global__ void embed_prep_kernel(const bf16* __restrict__ table, const int32_t* __restrict__ tokens,
                                  const bf16* __restrict__ rows, float* __restrict__ h, void* __restrict__ xg,
                                  size_t lo_off, int fmt, const float* __restrict__ g, float* __restrict__ ssq, int nt,
                                  int hidden, int vocab, int* status, float* __restrict__ amax, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) stamp_released(stamp);
  __shared__ float red[32];
  const int r = blockIdx.x;
  const bf16* src = tokens ? table + (size_t)checked_token(tokens, r, vocab, status) * hidden : rows + (size_t)r * hidden;
  float ss = 0.f, am = 0.f;
  for (int c = threadIdx.x; c < hidden; c += blockDim.x) {
    const float v = __bfloat162float(src[c]);
    h[(size_t)r * hidden + c] = v;
    store_act(xg, lo_off, (size_t)r * hidden + c, v * g[c], fmt);
    ss = fmaf(v, v, ss);
    am = fmaxf(am, abs_as_f16(v * g[c]));
  }
  ss = block_sum(ss, red);
  for (int t = threadIdx.x; t < nt; t += blockDim.x) ssq[(size_t)r * nt + t] = (t == 0) ? ss : 0.f;
  if (amax) {      // same layout as ssq: the whole row's maximum in slot 0
    __syncthreads();
    am = block_max(am, red);
    for (int t = threadIdx.x; t < nt; t += blockDim.x) amax[(size_t)r * nt + t] = (t == 0) ? am : 0.f;
  }
  if (threadIdx.x == 0) stamp_end(stamp);
}
void launch_embed_prep(const void* table, const int32_t* tokens, const void* rows, float* h, void* xg, size_t lo_off, int fmt,
                       const float* g, float* ssq, int nt, int n, int hidden, int vocab, int* status, cudaStream_t st, KStamp* stamp,
                       float* amax) {
  embed_prep_kernel<<<n, 256, 0, st>>>((const bf16*)table, tokens, (const bf16*)rows, h, xg, lo_off, fmt, g, ssq, nt, hidden, vocab,
                                       status, amax, stamp);
}

// bf16 rows -> f16 rows (saturating), for the operator-level entry points whose callers hand bf16 activations to an
// fp8-weight projection
__global__ void bf16_to_f16_kernel(const bf16* __restrict__ in, unsigned short* __restrict__ out, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = f16_bits_sat(__bfloat162float(in[i]));
}
void launch_bf16_to_f16(const void* in, void* out, size_t n, cudaStream_t st) {
  bf16_to_f16_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>((const bf16*)in, (unsigned short*)out, n);
}
// The same with one block per row, which also leaves amax[row] = max |f16 value| of the row: what the quantising
// projection takes its per-row scale from.
__global__ void bf16_rows_to_f16_amax_kernel(const bf16* __restrict__ in, unsigned short* __restrict__ out, int k,
                                             float* __restrict__ amax) {
  __shared__ float red[32];
  const size_t base = (size_t)blockIdx.x * k;
  float am = 0.f;
  for (int c = threadIdx.x; c < k; c += blockDim.x) {
    const unsigned short b = f16_bits_sat(__bfloat162float(in[base + c]));
    out[base + c] = b;
    am = fmaxf(am, fabsf(__half2float(__ushort_as_half(b))));
  }
  am = block_max(am, red);
  if (threadIdx.x == 0) amax[blockIdx.x] = am;
}
void launch_bf16_rows_to_f16_amax(const void* in, void* out, int m, int k, float* amax, cudaStream_t st) {
  bf16_rows_to_f16_amax_kernel<<<m, 256, 0, st>>>((const bf16*)in, (unsigned short*)out, k, amax);
}

// Sum of S split-K partials p[i * stride].  These kernels are a handful of dependent L2 round trips long, so every
// load that can be issued at once is: N loads in flight per call, added in index order (deterministic).
template <int N> struct Partials { float r[N]; };
template <int N>
__device__ __forceinline__ void issue_partials(Partials<N>& v, const float* __restrict__ p, size_t stride, int i0, int S) {
#pragma unroll
  for (int j = 0; j < N; ++j) v.r[j] = (i0 + j < S) ? __ldcg(p + (size_t)(i0 + j) * stride) : 0.f;
}
template <int N>
__device__ __forceinline__ float add_partials(const Partials<N>& v, float s) {
#pragma unroll
  for (int j = 0; j < N; ++j) s += v.r[j];
  return s;
}
// the partials from index i0 on, added to s
__device__ __forceinline__ float sum_partials_from(const float* __restrict__ p, size_t stride, int i0, int S, float s) {
  for (; i0 < S; i0 += 16) {
    Partials<16> v;
    issue_partials(v, p, stride, i0, S);
    s = add_partials(v, s);
  }
  return s;
}

// QKV finalisation: sum the split-K partials, apply the folded norm factor and the bias, rotate q and k
// (rotate-half pairs j, j + d/2), write q to its buffer and k, v into the layer's cache planes.
// grid (hq + 2 hkv heads, m rows), d/2 threads: thread j owns the pair (j, j + d/2) of one head.
template <typename T>
__global__ void fin_qkv_kernel(const float* __restrict__ part, int S, int m, const float2* __restrict__ cs,
                               const float* __restrict__ ssq, int nt, float inv_h, float eps,
                               const float* __restrict__ bq, const float* __restrict__ bk, const float* __restrict__ bv,
                               const float* __restrict__ sq, const float* __restrict__ sk, const float* __restrict__ sv,
                               T* __restrict__ q, T* __restrict__ kc, T* __restrict__ vc, int pos0, int hq, int hkv,
                               int d, int max_seq, const int* __restrict__ len_ptr, const float* __restrict__ amax_in,
                               float* __restrict__ amax_zero, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  const int head = blockIdx.x, r = blockIdx.y, j = threadIdx.x, half = d >> 1;
  // not written by any kernel of this forward: the cache length word, the scales and the biases
  if (len_ptr) pos0 = *len_ptr;
  float sc_a = 1.f, sc_b = 1.f, bi_a = 0.f, bi_b = 0.f;
  {
    const int hl = head < hq ? head : (head < hq + hkv ? head - hq : head - hq - hkv);
    const float* sc = head < hq ? sq : (head < hq + hkv ? sk : sv);
    const float* bi = head < hq ? bq : (head < hq + hkv ? bk : bv);
    if (sc) { sc_a = sc[hl * d + j]; sc_b = sc[hl * d + j + half]; }   // fp8 weights: per-output-channel factors
    if (bi) { bi_a = bi[hl * d + j]; bi_b = bi[hl * d + j + half]; }
  }
  pdl_wait();
  if (threadIdx.x == 0) stamp_released(stamp);
  __shared__ float s_rstd;
  // W8A8: the row's slot of the running maximum that this layer's gate/up epilogue raises; its last readers (the
  // previous layer's down projection) are long done, its next writers start after this kernel
  if (amax_zero && head == 0 && threadIdx.x == 0) amax_zero[r] = 0.f;
  // every load of this kernel is issued before the first result is needed
  const int width = (hq + 2 * hkv) * d;
  const size_t sstride = (size_t)m * width;
  const float* pa = part + (size_t)r * width + head * d + j;
  float ssq_v = 0.f, am = 0.f;
  if (threadIdx.x < 32) {
    for (int t = threadIdx.x; t < nt; t += 32) ssq_v += __ldcg(ssq + (size_t)r * nt + t);
    if (amax_in)     // W8A8: the partial sums are sums of code products; the row's scale joins the norm factor
      for (int t = threadIdx.x; t < nt; t += 32) am = fmaxf(am, __ldcg(amax_in + (size_t)r * nt + t));
  }
  const float2 c = (head < hq + hkv) ? __ldcg(&cs[r * half + j]) : make_float2(1.f, 0.f);
  Partials<16> va, vb;
  issue_partials(va, pa, sstride, 0, S);
  issue_partials(vb, pa + half, sstride, 0, S);
  if (threadIdx.x < 32) {
    // fixed order: lanes hold disjoint strided subsets, combined by the butterfly below
    const float t = warp_sum(ssq_v);
    am = warp_max(am);
    if (threadIdx.x == 0) s_rstd = rsqrtf(t * inv_h + eps) * (amax_in ? scale_of_amax(am) : 1.f);
  }
  float a = add_partials(va, 0.f), b = add_partials(vb, 0.f);
  a = sum_partials_from(pa, sstride, 16, S, a);
  b = sum_partials_from(pa + half, sstride, 16, S, b);
  __syncthreads();
  const float rstd = s_rstd;
  a = a * rstd * sc_a + bi_a;
  b = b * rstd * sc_b + bi_b;
  if (head < hq) {
    T* o = q + ((size_t)r * hq + head) * d;
    o[j] = from_f32<T>(a * c.x - b * c.y);
    o[j + half] = from_f32<T>(b * c.x + a * c.y);
  } else if (head < hq + hkv) {
    const int hk = head - hq;
    T* o = kc + ((size_t)hk * max_seq + pos0 + r) * d;
    o[j] = from_f32<T>(a * c.x - b * c.y);
    o[j + half] = from_f32<T>(b * c.x + a * c.y);
  } else {
    const int hk = head - hq - hkv;
    T* o = vc + ((size_t)hk * max_seq + pos0 + r) * d;
    o[j] = from_f32<T>(a);
    o[j + half] = from_f32<T>(b);
  }
  if (threadIdx.x == 0) stamp_end(stamp, true);
}
void launch_fin_qkv(const float* part, int S, int m, const float* cs, const float* ssq, int nt, int hidden, float eps,
                    const float* bq, const float* bk, const float* bv, const float* sq, const float* sk, const float* sv, void* q, void* kc, void* vc, int pos0, int hq,
                    int hkv, int d, int max_seq, int kv_type, cudaStream_t st, const int* len_ptr, KStamp* stamp, const float* amax_in,
                    float* amax_zero) {
  if (kv_type == KV_F16)
    launch_pdl(fin_qkv_kernel<__half>, dim3(hq + 2 * hkv, m), dim3(d / 2), 0, st, part, S, m, (const float2*)cs, ssq, nt, 1.f / (float)hidden,
               eps, bq, bk, bv, sq, sk, sv, (__half*)q, (__half*)kc, (__half*)vc, pos0, hq, hkv, d, max_seq, len_ptr, amax_in, amax_zero, stamp);
  else
    launch_pdl(fin_qkv_kernel<bf16>, dim3(hq + 2 * hkv, m), dim3(d / 2), 0, st, part, S, m, (const float2*)cs, ssq, nt, 1.f / (float)hidden,
               eps, bq, bk, bv, sq, sk, sv, (bf16*)q, (bf16*)kc, (bf16*)vc, pos0, hq, hkv, d, max_seq, len_ptr, amax_in, amax_zero, stamp);
}

// Residual finalisation: h += sum of split-K partials; xg = h * gain of the next norm (stored as `fmt`);
// ssq[row][tile] = sum of h^2 over the tile's 128 columns.  grid (nt tiles, m rows), 128 threads.
__global__ void __launch_bounds__(128) fin_resid_kernel(const float* __restrict__ part, int S, int m, int hidden,
                                                        float* __restrict__ h, const float* __restrict__ g,
                                                        void* __restrict__ xg, size_t lo_off, int fmt, float* __restrict__ ssq, int nt,
                                                        const float* __restrict__ scale, const float* __restrict__ amax_in,
                                                        int n_amax_in, float* __restrict__ amax_out, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  __shared__ float red[32];
  const int t = blockIdx.x, r = blockIdx.y, c = t * 128 + threadIdx.x;
  // weights (gain, scale) do not depend on the predecessor
  const float gc = (c < hidden) ? g[c] : 0.f;
  float sc = (c < hidden && scale) ? scale[c] : 1.f;
  pdl_wait();
  if (threadIdx.x == 0) stamp_released(stamp);
  // W8A8: the partial sums are sums of code products of a row quantised with the scale max / 448; the maxima are
  // asked for first and reduced only after the other loads are on their way
  float am_in = 0.f;
  if (amax_in) {
    if (n_amax_in == 1) am_in = __ldcg(amax_in + r);
    else for (int i = threadIdx.x; i < n_amax_in; i += 128) am_in = fmaxf(am_in, __ldcg(amax_in + (size_t)r * n_amax_in + i));
  }
  float v = 0.f;
  Partials<32> pv;
  float hv = 0.f;
  const size_t idx = (size_t)r * hidden + c, sstride = (size_t)m * hidden;
  if (c < hidden) {
    issue_partials(pv, part + idx, sstride, 0, S);
    hv = __ldcg(h + idx);
  }
  if (amax_in) sc *= scale_of_amax(n_amax_in == 1 ? am_in : block_max(am_in, red));
  if (c < hidden) {
    v = hv + sum_partials_from(part + idx, sstride, 32, S, add_partials(pv, 0.f)) * sc;
    h[idx] = v;
    store_act(xg, lo_off, idx, v * gc, fmt);
  }
  // one pass for the tile's sum of squares and (W8A8: the next projection's quantiser) the maximum of the stored xg
  __shared__ float red_s[4], red_m[4];
  {
    const float ws = warp_sum(v * v);
    const float wm = amax_out ? warp_max(c < hidden ? abs_as_f16(v * gc) : 0.f) : 0.f;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { red_s[threadIdx.x >> 5] = ws; red_m[threadIdx.x >> 5] = wm; }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    ssq[(size_t)r * nt + t] = (red_s[0] + red_s[2]) + (red_s[1] + red_s[3]);
    if (amax_out) amax_out[(size_t)r * nt + t] = fmaxf(fmaxf(red_m[0], red_m[1]), fmaxf(red_m[2], red_m[3]));
    stamp_end(stamp, true);
  }
}
void launch_fin_resid(const float* part, int S, int m, int hidden, float* h, const float* g, void* xg, size_t lo_off, int fmt,
                      float* ssq, int nt, const float* scale, cudaStream_t st, KStamp* stamp, const float* amax_in, int n_amax_in,
                      float* amax_out) {
  launch_pdl(fin_resid_kernel, dim3(nt, m), dim3(128), 0, st, part, S, m, hidden, h, g, xg, lo_off, fmt, ssq, nt, scale, amax_in,
             n_amax_in, amax_out, stamp);
}

// Merge the per-warp softmax statistics of the LM-head epilogue into confidence and prediction per row.
// stats[e * m + row] = (max, sum exp(l - max), argmax id) for e in [0, n_part).  grid m rows, 256 threads.
__global__ void __launch_bounds__(512) stats_merge_kernel(const float4* __restrict__ stats, int n_part, int m,
                                                          float* __restrict__ conf, int32_t* __restrict__ pred, KStamp* stamp) {
  if (threadIdx.x == 0) stamp_start(stamp);
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) stamp_released(stamp);
  __shared__ float sm_m[16], sm_s[16];
  __shared__ int sm_i[16];
  const int r = blockIdx.x;
  float mx = -INFINITY, s = 0.f;
  int ix = 0x7fffffff;
  auto merge = [&](float m2, float s2, int i2) {
    if (s2 == 0.f) return;
    if (s == 0.f) { mx = m2; s = s2; ix = i2; return; }
    const float mn = fmaxf(mx, m2);
    s = s * __expf(mx - mn) + s2 * __expf(m2 - mn);
    if (m2 > mx || (m2 == mx && i2 < ix)) ix = i2;
    mx = mn;
  };
  // ten loads in flight per thread: at the 3B / 7B vocabularies (4.7k partials per row) one L2 round trip in all
  for (int e0 = threadIdx.x; e0 < n_part; e0 += 10 * blockDim.x) {
    float4 v[10];
#pragma unroll
    for (int j = 0; j < 10; ++j) {
      const int e = e0 + j * blockDim.x;
      v[j] = e < n_part ? __ldcg(&stats[(size_t)e * m + r]) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < 10; ++j) merge(v[j].x, v[j].y, __float_as_int(v[j].z));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, mx, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    const int i2 = __shfl_xor_sync(0xffffffffu, ix, o);
    merge(m2, s2, i2);
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { sm_m[w] = mx; sm_s[w] = s; sm_i[w] = ix; }
  __syncthreads();
  if (threadIdx.x == 0) {
    mx = sm_m[0]; s = sm_s[0]; ix = sm_i[0];
    for (int k = 1; k < (int)(blockDim.x >> 5); ++k) merge(sm_m[k], sm_s[k], sm_i[k]);
    conf[r] = 1.f / s;
    pred[r] = ix;
    stamp_end(stamp);
  }
}
void launch_stats_merge(const void* stats, int n_part, int m, float* conf, int32_t* pred, cudaStream_t st, KStamp* stamp) {
  launch_pdl(stats_merge_kernel, dim3(m), dim3(512), 0, st, (const float4*)stats, n_part, m, conf, pred, stamp);
}

// ================================================================================================
// SwiGLU: act = silu(gate) * up, gu = [n, 2*inter] with gate in the first half of each row
// ================================================================================================
template <typename AT>
__global__ void swiglu_kernel(const float* __restrict__ gu, AT* __restrict__ act, int n, int inter) {
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)n * inter) return;
  int r = (int)(idx / inter), c = (int)(idx % inter);
  float g = gu[(size_t)r * 2 * inter + c], u = gu[(size_t)r * 2 * inter + inter + c];
  act[idx] = from_f32<AT>(g / (1.f + expf(-g)) * u);
}
void launch_swiglu(const float* gu, void* act, int n, int inter, int dtype, cudaStream_t st) {
  size_t total = (size_t)n * inter;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (dtype == DT_F32) swiglu_kernel<float><<<blocks, 256, 0, st>>>(gu, (float*)act, n, inter);
  else swiglu_kernel<bf16><<<blocks, 256, 0, st>>>(gu, (bf16*)act, n, inter);
}

// ================================================================================================
// confidence and prediction of a row: pred = argmax_{v != mask_id} l_v (lowest id on a tie),
// conf = 1 / sum_{v != mask_id} exp(l_v - l_pred)
// ================================================================================================
__global__ void __launch_bounds__(1024) row_stats_kernel(const float* __restrict__ logits, int vocab, int mask_id,
                                                       float* __restrict__ conf, int32_t* __restrict__ pred) {
  __shared__ float red[32];
  __shared__ float smax[32];
  __shared__ int sidx[32];
  const float* l = logits + (size_t)blockIdx.x * vocab;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int v = threadIdx.x; v < vocab; v += blockDim.x) {
    if (v == mask_id) continue;
    float x = l[v];
    if (x > best) { best = x; bi = v; }
  }
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float ob = __shfl_xor_sync(0xffffffffu, best, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
  }
  if (lane == 0) { smax[w] = best; sidx[w] = bi; }
  __syncthreads();
  if (w == 0) {
    best = lane < nw ? smax[lane] : -INFINITY;
    bi = lane < nw ? sidx[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ob = __shfl_xor_sync(0xffffffffu, best, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    if (lane == 0) { smax[0] = best; sidx[0] = bi; }
  }
  __syncthreads();
  best = smax[0];
  float s = 0.f;
  for (int v = threadIdx.x; v < vocab; v += blockDim.x)
    if (v != mask_id) s += __expf(l[v] - best);
  s = block_sum(s, red);
  if (threadIdx.x == 0) { conf[blockIdx.x] = 1.f / s; pred[blockIdx.x] = sidx[0]; }
}
void launch_row_stats(const float* logits, int n, int vocab, int mask_id, float* conf, int32_t* pred, cudaStream_t st) {
  row_stats_kernel<<<n, 1024, 0, st>>>(logits, vocab, mask_id, conf, pred);
}

// ================================================================================================
// unmask selection (one CTA of 64 threads; n <= 64)
// ================================================================================================
__global__ void select_kernel(const float* __restrict__ conf, const int32_t* __restrict__ pred,
                              int32_t* __restrict__ tokens, uint8_t* __restrict__ masked,
                              uint8_t* __restrict__ unmask, int32_t* __restrict__ info, int n, int rule,
                              float threshold, int k, int shift, cudaGraphConditionalHandle cond, int loop) {
  pdl_trigger();
  pdl_wait();
  __shared__ float c[64];
  __shared__ int mk[64];
  int i = threadIdx.x;
  // shift = 1: position i is predicted by row i - 1; position 0 has no predictor and is never selected
  c[i] = (i < n && i >= shift) ? conf[i - shift] : -1.f;
  mk[i] = (i < n && i >= shift) ? (int)masked[i] : 0;
  // a masked position 0 under shift = 1 has no predictor: nothing is revealed and it is reported as remaining
  const int stuck = (shift && n > 0 && masked[0]) ? 1 : 0;
  __syncthreads();
  int is_m = mk[i];
  int rank = 0, n_masked = 0;
  for (int j = 0; j < n; ++j) {
    if (!mk[j]) continue;
    ++n_masked;
    if (c[j] > c[i] || (c[j] == c[i] && j < i)) ++rank;
  }
  int sel;
  if (rule == 0) {
    int hit = is_m && (c[i] > threshold);
    int any = __syncthreads_or(hit);
    sel = any ? hit : (is_m && rank == 0);
  } else {
    sel = is_m && rank < k;
  }
  if (stuck) sel = 0;
  int n_sel = __syncthreads_count(sel);
  if (i < n) {
    unmask[i] = (uint8_t)sel;
    if (sel) { tokens[i] = pred[i - shift]; masked[i] = 0; }
  }
  if (i == 0) {
    const int left = n_masked - n_sel + stuck;
    info[0] = n_sel; info[1] = left; info[2] = info[2] + 1;
    if (loop) {
      // body of the on-device decode loop: run another denoise step while masked positions are left.  Every step
      // reveals at least one position, so the loop ends after at most n steps; the explicit count is a second bound.
      const int it = info[5] + 1;
      info[5] = it;
      cudaGraphSetConditional(cond, (left > 0 && n_sel > 0 && it < n) ? 1u : 0u);
    }
  }
}
void launch_select(const float* conf, const int32_t* pred, int32_t* tokens, uint8_t* masked, uint8_t* unmask,
                   int32_t* info, int n, int rule, float threshold, int k, cudaStream_t st, int shift,
                   cudaGraphConditionalHandle cond, int loop) {
  select_kernel<<<1, 64, 0, st>>>(conf, pred, tokens, masked, unmask, info, n, rule, threshold, k, shift, cond, loop);
}

// Longest accepted prefix of a drafted block d against the causal predictions a (a[j] predicts the token after d[j]):
// k = 1 + (first j in [0, n-2] with a[j] != d[j+1]; n-1 if none).  out = {k, a[k-1]}.
__global__ void accept_kernel(const int32_t* __restrict__ a, const int32_t* __restrict__ d, int n, int32_t* __restrict__ out) {
  __shared__ int first;
  if (threadIdx.x == 0) first = n - 1;
  __syncthreads();
  const int j = threadIdx.x;
  if (j < n - 1 && a[j] != d[j + 1]) atomicMin(&first, j);
  __syncthreads();
  if (threadIdx.x == 0) { out[0] = first + 1; out[1] = a[first]; }
}
void launch_accept(const int32_t* a, const int32_t* d, int n, int32_t* out, cudaStream_t st) {
  accept_kernel<<<1, 64, 0, st>>>(a, d, n, out);
}

// Read-only streaming of a buffer: every CTA walks its share with 16-byte loads, eight in flight per thread, and folds
// what it reads into one word (so that the loads cannot be dropped).  A yardstick for the read bandwidth a kernel of this
// library can reach at all; no part of the decoding path.
__global__ void __launch_bounds__(256) stream_read_kernel(const uint4* __restrict__ buf, size_t n16, unsigned* __restrict__ sink) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  unsigned acc = 0;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldcs(buf + i + u * stride);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += stride) { const uint4 v = __ldcs(buf + i); acc ^= v.x ^ v.y ^ v.z ^ v.w; }
  if (acc == 0x9e3779b9u) atomicAdd(sink, 1u);     // practically never: keeps the loads alive without a store per thread
}
void launch_stream_read(const void* buf, size_t bytes, unsigned* sink, int ctas, cudaStream_t st) {
  stream_read_kernel<<<ctas, 256, 0, st>>>((const uint4*)buf, bytes / 16, sink);
}

// ---- quadratic self-speculative decoding (Appendix B, Alg. 2) --------------------------------------------------------
// Row order of the B (B + 1) rows of one forward: rows 0 .. B-1 are the draft tokens d_0 .. d_{B-1} (the first tokens of
// the groups), row B + i B + (j - 1) is mask token j (1 <= j <= B) of group i.  With the first tokens in front, the rows
// whose K / V outlive the forward ("keep every (B+1)-th entry", and of those the accepted ones) are the first k staging
// rows of the cache.
//   pos_off[r]: position id minus the position of d_0: i for a first token, i + j for a mask token
//   mask[r]   : bit r' = row r reads row r'.  (b) first token i reads first tokens <= i; (c) a mask token of group i reads
//               its group's first token and all its mask tokens; (d) nothing else -- chain != 0: also the first tokens of
//               the groups before i.
__global__ void quad_layout_kernel(int B, int chain, unsigned long long* __restrict__ mask, int* __restrict__ pos_off) {
  const int r = threadIdx.x, n = B * (B + 1);
  if (r >= n) return;
  if (r < B) {
    mask[r] = (2ull << r) - 1ull;                              // bits 0 .. r
    pos_off[r] = r;
  } else {
    const int i = (r - B) / B, j = (r - B) % B + 1;
    const unsigned long long group = ((B == 64 ? 0ull : (1ull << B)) - 1ull) << (B + i * B);   // its B mask rows
    unsigned long long m = group | (1ull << i);
    if (chain) m |= (1ull << i) - 1ull;
    mask[r] = m;
    pos_off[r] = i + j;
  }
}
void launch_quad_layout(int B, int chain, unsigned long long* mask, int* pos_off, cudaStream_t st) {
  quad_layout_kernel<<<1, 64, 0, st>>>(B, chain, mask, pos_off);
}
// tokens of the rows above from the draft d
__global__ void quad_build_kernel(const int32_t* __restrict__ d, int B, int mask_id, int32_t* __restrict__ tokens,
                                  uint8_t* __restrict__ masked) {
  const int r = threadIdx.x;
  if (r >= B * (B + 1)) return;
  tokens[r] = r < B ? d[r] : mask_id;
  masked[r] = r >= B;
}
void launch_quad_build(const int32_t* d, int B, int mask_id, int32_t* tokens, uint8_t* masked, cudaStream_t st) {
  quad_build_kernel<<<1, 64, 0, st>>>(d, B, mask_id, tokens, masked);
}
// Alg. 2 step 1: d_0 = the token the prompt's last row predicts, d_i = prediction of mask row i - 1 (shift by one)
__global__ void quad_first_draft_kernel(const int32_t* __restrict__ pred, int32_t first, int B, int32_t* __restrict__ d) {
  const int i = threadIdx.x;
  if (i < B) d[i] = i == 0 ? first : pred[i - 1];
}
void launch_quad_first_draft(const int32_t* pred, int32_t first, int B, int32_t* d, cudaStream_t st) {
  quad_first_draft_kernel<<<1, 64, 0, st>>>(pred, first, B, d);
}
// Alg. 2's verify loop on the predictions of one forward (P_{i,0} = pred[i], P_{i,j} = pred[B + i B + j - 1]):
// k = 1; while k < B and P_{k-1,0} = d_k: k += 1.  accepted[0 .. k) = d_0 .. d_{k-1}; d <- P_{k-1,1..B}; out = {k}.
__global__ void quad_accept_kernel(const int32_t* __restrict__ pred, int32_t* __restrict__ d, int B, int32_t* __restrict__ accepted,
                                   int32_t* __restrict__ out) {
  __shared__ int k_s;
  __shared__ int32_t old_d[64];
  const int t = threadIdx.x;
  if (t < B) old_d[t] = d[t];
  __syncthreads();
  if (t == 0) {
    int k = 1;
    while (k < B && pred[k - 1] == old_d[k]) ++k;
    k_s = k;
    out[0] = k;
  }
  __syncthreads();
  const int k = k_s;
  if (t < B) {
    if (accepted) accepted[t] = t < k ? old_d[t] : -1;
    d[t] = pred[B + (k - 1) * B + t];
  }
}
void launch_quad_accept(const int32_t* pred, int32_t* d, int B, int32_t* accepted, int32_t* out, cudaStream_t st) {
  quad_accept_kernel<<<1, 64, 0, st>>>(pred, d, B, accepted, out);
}

// Commit of the finished block (Bc rows) and opening of the next one (Bn rows) for ONE forward over Bc + Bn rows:
// rows = [finished tokens ; next block's initial tokens]; mask: a finished row reads the finished rows up to itself
// (Alg. 1 verify mask), a row of the next block reads every row (the committed block is part of its context, its own
// block is bidirectional); the block state becomes the next block's.
__global__ void fuse_begin_kernel(int32_t* __restrict__ blk_tokens, uint8_t* __restrict__ blk_masked, int Bc,
                                  const int32_t* __restrict__ init, int Bn, int mask_id, int32_t* __restrict__ rows,
                                  unsigned long long* __restrict__ mask, int32_t* __restrict__ info) {
  __shared__ int32_t nxt[64];
  const int i = threadIdx.x, n = Bc + Bn;
  const int32_t old = i < Bc ? blk_tokens[i] : 0;
  nxt[i] = (i < Bn && init) ? init[i] : mask_id;
  __syncthreads();
  if (i < n) {
    rows[i] = i < Bc ? old : nxt[i - Bc];
    mask[i] = i < Bc ? (2ull << i) - 1ull : (n == 64 ? ~0ull : (1ull << n) - 1ull);
  }
  const int m = (i < Bn) && (nxt[i] == mask_id);
  if (i < Bn) { blk_tokens[i] = nxt[i]; blk_masked[i] = (uint8_t)m; }
  const int cnt = __syncthreads_count(m);
  if (i == 0) { info[0] = 0; info[1] = cnt; info[2] = 0; }
}
void launch_fuse_begin(int32_t* blk_tokens, uint8_t* blk_masked, int Bc, const int32_t* init, int Bn, int mask_id, int32_t* rows,
                       unsigned long long* mask, int32_t* info, cudaStream_t st) {
  fuse_begin_kernel<<<1, 64, 0, st>>>(blk_tokens, blk_masked, Bc, init, Bn, mask_id, rows, mask, info);
}

__global__ void init_block_kernel(int32_t* tokens, uint8_t* masked, int32_t* info, const int32_t* init, int n, int mask_id,
                                  int step) {
  int i = threadIdx.x;
  int t = (i < n && init) ? init[i] : mask_id;
  int m = (i < n) && (t == mask_id);
  if (i < n) { tokens[i] = t; masked[i] = (uint8_t)m; }
  int cnt = __syncthreads_count(m);
  if (i == 0) { info[0] = 0; info[1] = cnt; info[2] = step; }
}
void launch_init_block(int32_t* tokens, uint8_t* masked, int32_t* info, const int32_t* init, int n, int mask_id, int step,
                       cudaStream_t st) {
  init_block_kernel<<<1, 64, 0, st>>>(tokens, masked, info, init, n, mask_id, step);
}

// ================================================================================================
// attention, CUDA-core version: one CTA per (query head, row).  Exact-fp32 path of the fp32
// configuration and the fallback where the tensor-core kernel does not apply.
// ================================================================================================
template <typename AT>
__global__ void __launch_bounds__(128) attn_simt_kernel(const AT* __restrict__ q, const AT* __restrict__ kc,
                                                        const AT* __restrict__ vc, AT* __restrict__ out, int n,
                                                        int L, int max_seq, int hq, int hkv, int d, int causal,
                                                        const unsigned long long* __restrict__ row_mask) {
  extern __shared__ float smem[];
  float* qs = smem;          // [d]
  float* red = smem + d;     // [32]
  float* ov = red + 32;      // [128]
  float* sc = ov + 128;      // [T]
  const int hqi = blockIdx.x, r = blockIdx.y;
  const int hk = hqi / (hq / hkv);
  const int T = causal ? (L + r + 1) : (L + n);
  const float scale = rsqrtf((float)d);
  const AT* qrow = q + ((size_t)r * hq + hqi) * d;
  for (int t = threadIdx.x; t < d; t += blockDim.x) qs[t] = to_f32(qrow[t]) * scale;
  __syncthreads();
  const AT* kbase = kc + (size_t)hk * max_seq * d;
  const AT* vbase = vc + (size_t)hk * max_seq * d;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int epl = d / 32;
  for (int j = w; j < T; j += nw) {
    const AT* kr = kbase + (size_t)j * d + lane * epl;
    float p = 0.f;
    for (int e = 0; e < epl; ++e) p = fmaf(qs[lane * epl + e], to_f32(kr[e]), p);
    p = warp_sum(p);
    // explicit mask among the n rows: bit r' of row_mask[r] = row r reads row r' (the cache is always read)
    if (row_mask && j >= L && !((row_mask[r] >> (j - L)) & 1ull)) p = -INFINITY;
    if (lane == 0) sc[j] = p;
  }
  __syncthreads();
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < T; j += blockDim.x) mx = fmaxf(mx, sc[j]);
  mx = block_max(mx, red);
  float sum = 0.f;
  for (int j = threadIdx.x; j < T; j += blockDim.x) { float e = expf(sc[j] - mx); sc[j] = e; sum += e; }
  sum = block_sum(sum, red);
  __syncthreads();
  const int dd = threadIdx.x % d, part = threadIdx.x / d, nparts = blockDim.x / d;
  float acc = 0.f;
  for (int j = part; j < T; j += nparts) acc = fmaf(sc[j], to_f32(vbase[(size_t)j * d + dd]), acc);
  ov[threadIdx.x] = acc;
  __syncthreads();
  if (part == 0) {
    for (int p2 = 1; p2 < nparts; ++p2) acc += ov[p2 * d + dd];
    out[((size_t)r * hq + hqi) * d + dd] = from_f32<AT>(acc / sum);
  }
}

int launch_attention_simt(const AttnArgs& a, cudaStream_t st, cudaError_t* err) {
  size_t smem = (size_t)(a.d + 32 + 128 + a.cache_len + a.n) * sizeof(float);
  dim3 grid(a.hq, a.n);
  *err = cudaSuccess;
  if (a.dtype == DT_F32) {
    if (smem > 48 * 1024) *err = cudaFuncSetAttribute(attn_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (*err != cudaSuccess) return -1;
    attn_simt_kernel<float><<<grid, 128, smem, st>>>((const float*)a.q, (const float*)a.kc, (const float*)a.vc,
                                                     (float*)a.out, a.n, a.cache_len, a.max_seq, a.hq, a.hkv, a.d, a.causal, a.row_mask);
  } else {
    if (smem > 48 * 1024) *err = cudaFuncSetAttribute(attn_simt_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (*err != cudaSuccess) return -1;
    attn_simt_kernel<bf16><<<grid, 128, smem, st>>>((const bf16*)a.q, (const bf16*)a.kc, (const bf16*)a.vc, (bf16*)a.out,
                                                    a.n, a.cache_len, a.max_seq, a.hq, a.hkv, a.d, a.causal, a.row_mask);
  }
  *err = cudaGetLastError();
  return *err == cudaSuccess ? 1 : -1;
}

}  // namespace fdk
