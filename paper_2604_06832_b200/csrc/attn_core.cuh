// Core of the split-KV, block-masked GQA attention (bf16 or f16 operands, mma.sync m16n8k16, online softmax in
// fp32).  T is the element type of q and of the KV cache; the probabilities are rounded to T for the P.V product.
#pragma once
#include "common.cuh"

namespace fdk {

constexpr int AT_ROWS = 64;    // query rows per CTA (4 warps x 16)
constexpr int AT_KEYS = 64;    // keys per shared-memory tile
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
template <typename T> __device__ __forceinline__ void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1);
template <> __device__ __forceinline__ void mma_16816<bf16>(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <> __device__ __forceinline__ void mma_16816<__half>(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <typename T> __device__ __forceinline__ uint32_t pack2(float lo, float hi);
template <> __device__ __forceinline__ uint32_t pack2<bf16>(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
template <> __device__ __forceinline__ uint32_t pack2<__half>(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);       // probabilities lie in [0, 1]: no range concern
  return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a swizzled [rows][D] bf16 tile
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

// Split of T keys into chunks of whole 64-key tiles, at most `bound` chunks (the same on host and device, so a launch
// whose grid was sized for `bound` can take the sequence length from device memory).
__host__ __device__ inline void attn_chunking(int T, int bound, int* chunk_keys, int* n_chunks) {
  const int tiles = (T + AT_KEYS - 1) / AT_KEYS;
  int want = bound < tiles ? bound : tiles;
  if (want < 1) want = 1;
  *chunk_keys = ((tiles + want - 1) / want) * AT_KEYS;
  *n_chunks = (T + *chunk_keys - 1) / *chunk_keys;
}

// Barrier of the 128 threads that work on one attention item (named barrier 1, so the threads may be a
// subset of a larger CTA).
__device__ __forceinline__ void attn_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// One attention work item: the query heads [hk * G + grp * qh, +qh) of KV head hk against the keys of `chunk`.
// Called by 128 threads (tid 0..127) that own attn_smem_bytes<D>() bytes of shared memory at address sQ (128-byte
// aligned).  Leaves the unnormalised partial (O, running max, running sum) of every row in part_o / part_ml.
// PDL: the caller is a kernel launched with programmatic dependent launch that has not yet waited for its predecessor
// (which writes q and the K/V rows of positions >= L); a first key tile that lies wholly in the committed cache is
// then requested before that wait.
template <int D, typename E, bool PDL = false>
__device__ __forceinline__ void attn_item(const E* q, const E* kc, const E* vc, float* part_o, float2* part_ml,
                                          int n, int L, int max_seq, int hq, int hkv, int qh, int chunk_keys, int n_chunks,
                                          int causal, int chunk, int grp, int hk, uint32_t sQ, int tid) {
  constexpr int CH = D / 8;                 // 16-byte chunks per row
  constexpr int TILE_BYTES = AT_KEYS * D * 2;
  const uint32_t sK = sQ + AT_ROWS * D * 2;            // 2 buffers
  const uint32_t sV = sK + 2 * TILE_BYTES;             // 2 buffers
  const int G = hq / hkv;
  const int head0 = hk * G + grp * qh;                 // first query head of this CTA
  const int heads_here = min(qh, G - grp * qh);
  const int m_valid = heads_here * n;
  const int T = L + n;
  const int key_begin = chunk * chunk_keys;
  const int key_end = min(T, key_begin + chunk_keys);
  const int n_tiles = (key_end - key_begin + AT_KEYS - 1) / AT_KEYS;
  const int warp = tid >> 5, lane = tid & 31;
  const E* kbase = kc + (size_t)hk * max_seq * D;
  const E* vbase = vc + (size_t)hk * max_seq * D;

  auto load_tile = [&](int t, int buf) {
    const int j0 = key_begin + t * AT_KEYS;
    for (int v = tid; v < AT_KEYS * CH; v += 128) {
      const int r = v / CH, c = v % CH;
      const int j = j0 + r;
      const bool ok = j < key_end;
      const size_t off = (size_t)(ok ? j : 0) * D + c * 8;
      cp_async16(sK + buf * TILE_BYTES + swz<D>(r, c), kbase + off, ok ? 16 : 0);
      cp_async16(sV + buf * TILE_BYTES + swz<D>(r, c), vbase + off, ok ? 16 : 0);
    }
  };
  const bool early = PDL && n_tiles > 0 && key_begin + AT_KEYS <= L;
  if (early) load_tile(0, 0);
  // ---- stage Q (rows = heads_here x n; row r -> head r / n, token r % n); addresses worked out before the wait ----
  constexpr int QV = AT_ROWS * CH / 128;
  const E* q_src[QV];
  uint32_t q_dst[QV];
#pragma unroll
  for (int u = 0; u < QV; ++u) {
    const int v = tid + u * 128;
    const int r = v / CH, c = v % CH;
    const bool ok = r < m_valid;
    const int hl = ok ? r / n : 0, i = ok ? r % n : 0;
    q_src[u] = ok ? q + ((size_t)i * hq + head0 + hl) * D + c * 8 : nullptr;
    q_dst[u] = sQ + swz<D>(r, c);
  }
  if (PDL) pdl_wait();
#pragma unroll
  for (int u = 0; u < QV; ++u) cp_async16(q_dst[u], q_src[u] ? q_src[u] : q, q_src[u] ? 16 : 0);
  if (n_tiles > 0 && !early) load_tile(0, 0);
  cp_async_commit();

  const int row0 = warp * 16;                       // this warp's rows of the CTA tile
  const bool warp_live = row0 < m_valid;
  const int g = lane >> 2, tq = lane & 3;
  const int r_lo = row0 + g, r_hi = r_lo + 8;       // the two rows this thread owns
  // last visible key (exclusive) of each row
  const int lim_lo = (r_lo < m_valid) ? (causal ? L + (r_lo % n) + 1 : T) : 0;
  const int lim_hi = (r_hi < m_valid) ? (causal ? L + (r_hi % n) + 1 : T) : 0;
  const float sl2 = rsqrtf((float)D) * LOG2E;       // scores kept in the log2 domain

  uint32_t qf[D / 16][4];
  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

  for (int t = 0; t < n_tiles; ++t) {
    const int buf = t & 1;
    if (t + 1 < n_tiles) load_tile(t + 1, buf ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    attn_bar();
    if (t == 0) {
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk)
        ldsm_x4(sQ + swz<D>(row0 + (lane & 15), kk * 2 + (lane >> 4)), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
    }
    if (warp_live) {
      float s[AT_KEYS / 8][4];
#pragma unroll
      for (int i = 0; i < AT_KEYS / 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
      const uint32_t kt = sK + buf * TILE_BYTES;
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
        for (int np = 0; np < AT_KEYS / 16; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(kt + swz<D>(np * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
          mma_16816<E>(s[2 * np], qf[kk], b0, b1);
          mma_16816<E>(s[2 * np + 1], qf[kk], b2, b3);
        }
      }
      // mask + running max
      const int j0 = key_begin + t * AT_KEYS;
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < AT_KEYS / 8; ++nt) {
        const int j = j0 + nt * 8 + tq * 2;
        s[nt][0] = (j < lim_lo) ? s[nt][0] * sl2 : -INFINITY;
        s[nt][1] = (j + 1 < lim_lo) ? s[nt][1] * sl2 : -INFINITY;
        s[nt][2] = (j < lim_hi) ? s[nt][2] * sl2 : -INFINITY;
        s[nt][3] = (j + 1 < lim_hi) ? s[nt][3] * sl2 : -INFINITY;
        mx_lo = fmaxf(mx_lo, fmaxf(s[nt][0], s[nt][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(s[nt][2], s[nt][3]));
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float ref_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, ref_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
      const float al_lo = exp2f(m_lo - ref_lo), al_hi = exp2f(m_hi - ref_hi);   // exp2(-inf) = 0 on the first tile
      m_lo = mn_lo; m_hi = mn_hi;
      float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
      for (int nt = 0; nt < AT_KEYS / 8; ++nt) {
        s[nt][0] = exp2f(s[nt][0] - ref_lo); s[nt][1] = exp2f(s[nt][1] - ref_lo);
        s[nt][2] = exp2f(s[nt][2] - ref_hi); s[nt][3] = exp2f(s[nt][3] - ref_hi);
        sum_lo += s[nt][0] + s[nt][1];
        sum_hi += s[nt][2] + s[nt][3];
      }
      l_lo = l_lo * al_lo + sum_lo;
      l_hi = l_hi * al_hi + sum_hi;
#pragma unroll
      for (int i = 0; i < D / 8; ++i) { o[i][0] *= al_lo; o[i][1] *= al_lo; o[i][2] *= al_hi; o[i][3] *= al_hi; }
      const uint32_t vt = sV + buf * TILE_BYTES;
#pragma unroll
      for (int kk = 0; kk < AT_KEYS / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack2<E>(s[2 * kk][0], s[2 * kk][1]);
        pa[1] = pack2<E>(s[2 * kk][2], s[2 * kk][3]);
        pa[2] = pack2<E>(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        pa[3] = pack2<E>(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int dp = 0; dp < D / 16; ++dp) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(vt + swz<D>(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)), b0, b1, b2, b3);
          mma_16816<E>(o[2 * dp], pa, b0, b1);
          mma_16816<E>(o[2 * dp + 1], pa, b2, b3);
        }
      }
    }
    attn_bar();
  }
  cp_async_wait<0>();

  // ---- partial results: the quad's four lanes hold the row sums in pieces ----
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int r = half ? r_hi : r_lo;
    if (r >= m_valid) continue;
    const int head = head0 + r / n, i = r % n;
    const size_t slot = ((size_t)head * n + i) * n_chunks + chunk;
    float* dst = part_o + slot * D;
#pragma unroll
    for (int dt = 0; dt < D / 8; ++dt) {
      float2 v = half ? make_float2(o[dt][2], o[dt][3]) : make_float2(o[dt][0], o[dt][1]);
      *reinterpret_cast<float2*>(dst + dt * 8 + tq * 2) = v;
    }
    if (tq == 0) part_ml[slot] = half ? make_float2(m_hi, l_hi) : make_float2(m_lo, l_lo);
  }
  attn_bar();   // the shared-memory tiles may be reused by the caller's next item
}

template <int D> constexpr int attn_smem_bytes() { return AT_ROWS * D * 2 + 4 * AT_KEYS * D * 2; }


// Merge of the key chunks of one (row, head) by one warp: out = sum_c w_c O_c / sum_c w_c l_c, w_c = 2^(m_c - max m).
// Lane j owns D / 32 consecutive output features; the chunk statistics are spread over the lanes.
// The result is stored as `fmt` (XF_*) at element offset out_idx of `out`.
template <int D>
__device__ __forceinline__ void attn_merge_warp(const float* att_o, const float2* att_ml, void* out, size_t out_idx, size_t lo_off,
                                                int fmt, size_t slot0, int n_chunks, int lane) {
  constexpr int VPL = D / 32;
  constexpr int CB = 16;     // chunks whose partial outputs are in flight together
  // The statistics and the first CB partial outputs are requested together: one L2 round trip for up to 16 chunks.
  float2 ml0 = make_float2(-INFINITY, 0.f);
  if (lane < n_chunks) ml0 = __ldcg(&att_ml[slot0 + lane]);
  float ov[CB][VPL];
  auto issue = [&](int c0) {
#pragma unroll
    for (int cc = 0; cc < CB; ++cc) {
      const float* src = att_o + (slot0 + c0 + cc) * D + lane * VPL;
      if (c0 + cc < n_chunks) {
        if (VPL == 4) {
          const float4 o = __ldcg(reinterpret_cast<const float4*>(src));
          ov[cc][0] = o.x; ov[cc][1] = o.y; ov[cc][2] = o.z; ov[cc][VPL - 1] = o.w;
        } else {
          const float2 o = __ldcg(reinterpret_cast<const float2*>(src));
          ov[cc][0] = o.x; ov[cc][VPL - 1] = o.y;
        }
      } else {
#pragma unroll
        for (int i = 0; i < VPL; ++i) ov[cc][i] = 0.f;
      }
    }
  };
  issue(0);
  float mx = ml0.x;
  for (int c = lane + 32; c < n_chunks; c += 32) mx = fmaxf(mx, __ldcg(&att_ml[slot0 + c]).x);
  mx = warp_max(mx);
  float den = 0.f, acc[VPL];
#pragma unroll
  for (int i = 0; i < VPL; ++i) acc[i] = 0.f;
  for (int c0 = 0; c0 < n_chunks; c0 += 32) {
    const int c = c0 + lane;
    float w = 0.f;
    if (c < n_chunks) {
      const float2 ml = (c0 == 0) ? ml0 : __ldcg(&att_ml[slot0 + c]);
      if (ml.y != 0.f) { w = exp2f(ml.x - mx); den = fmaf(w, ml.y, den); }
    }
    for (int h0 = 0; h0 < 32 && c0 + h0 < n_chunks; h0 += CB) {
      if (c0 + h0 > 0) issue(c0 + h0);
#pragma unroll
      for (int cc = 0; cc < CB; ++cc) {
        const float wc = __shfl_sync(0xffffffffu, w, h0 + cc);     // zero for chunks past the end
#pragma unroll
        for (int i = 0; i < VPL; ++i) acc[i] = fmaf(wc, ov[cc][i], acc[i]);
      }
    }
  }
  den = warp_sum(den);
  const float inv = 1.f / den;
#pragma unroll
  for (int i = 0; i < VPL; ++i) store_act(out, lo_off, out_idx + lane * VPL + i, acc[i] * inv, fmt);
}

}  // namespace fdk
