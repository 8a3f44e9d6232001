// Split-KV, block-masked GQA attention for the tensor-core path (Sec. 3.3 masks; Alg. 1 draft / verify).
//
// One CTA = (KV head, group of query heads that share it, chunk of keys).  The CTA's rows are the block's n rows of
// each of its query heads (ROWS = 64 or 128 in all, 16 per compute warp).  The K and V tiles of the chunk (64 keys
// each) are fetched by one producer thread with 2-D TMA loads (128-byte swizzle) into a ring of shared-memory stages
// guarded by full / empty mbarriers; tiles that lie wholly in the committed cache are requested before the wait for
// the predecessor kernel.  Scores and P.V run on mma.sync m16n8k16 (bf16 or f16 operands, fp32 accumulate) with an
// online softmax in fp32; each CTA leaves an unnormalised partial (O, running max, running sum) and a small second
// kernel merges the chunks.  The in-block mask is applied by key index: denoise rows see all L + n keys, commit /
// prefill rows see keys <= L + i.  Two shapes of CTA: 64 rows with a two-stage ring, two CTAs per SM (short caches:
// one or two tiles per CTA); 128 rows with up to six tiles resident at once, one CTA per SM (long caches: every K/V
// byte crosses from L2 half as often and the whole chunk is in flight from the start).
// Every mbarrier wait is bounded; a wait that gives up records ST_ATTENTION in the status word and the CTA drains its
// copies in flight and returns.
#include "attn_plan.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace fdk {


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

// byte offset of 16-byte chunk `chunk` of row `row` in the Q tile: rows of D * 2 bytes, chunks XOR-swizzled by row
template <int D>
__device__ __forceinline__ uint32_t swz_q(int row, int chunk) {
  return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}
// the same for a K or V tile as the TMA leaves it: one [64 keys][128 bytes] sub-tile per 64 head dimensions, 16-byte
// chunks XOR-swizzled by the key's row (the 128-byte swizzle of the tensor map)
__device__ __forceinline__ uint32_t swz_kv(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * (AT_KEYS * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int D, int ROWS>
struct AtSmem {
  static constexpr int STAGES = ROWS == 64 ? 2 : (D == 128 ? 6 : 12);
  static constexpr int Q_BYTES = ROWS * D * 2;
  static constexpr int TILE_BYTES = AT_KEYS * D * 2;          // one K or one V tile
  static constexpr int STAGE_BYTES = 2 * TILE_BYTES;          // K then V
  static constexpr int BAR_OFF = Q_BYTES + STAGES * STAGE_BYTES;
  static constexpr int TOTAL = BAR_OFF + 8 * (2 * STAGES) + 16 + 1024;   // barriers, abort flag, alignment slack
  static constexpr int THREADS = (ROWS / 16) * 32 + 32;       // compute warps + the producer warp
};

struct AttnParams {
  CUtensorMap tm_k, tm_v;     // [Hkv * max_seq, D] views of the layer's K and V planes, box {64, 64}
  const void* q;              // [n, Hq, D]
  float* part_o;              // [Hq][n][chunks][D]
  float2* part_ml;            // [Hq][n][chunks]
  int n, L, max_seq, hq, hkv, qh, chunk_keys, n_chunks, causal;
  const int* len_ptr;         // nullable: the cache length is read from device memory and the chunking derived from it
  const unsigned long long* row_mask;   // nullable: bit r' of word r = row r reads row r' of this forward (AttnArgs::row_mask)
  int* status;                // nullable: status words (see TcOut::status)
  KStamp* stamp;
};

template <int D, typename E, int ROWS>
__global__ void __launch_bounds__(AtSmem<D, ROWS>::THREADS, ROWS == 64 ? 2 : 1) attn_mma_kernel(const __grid_constant__ AttnParams p) {
  using S = AtSmem<D, ROWS>;
  constexpr int CH = D / 8;                 // 16-byte chunks per row
  constexpr int NW = ROWS / 16;             // compute warps
  constexpr int NCT = NW * 32;              // compute threads
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sQ = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (sQ - raw);
  const uint32_t sKV = sQ + S::Q_BYTES;
  const uint32_t bar0 = sQ + S::BAR_OFF;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (S::STAGES + s); };
  volatile int* abort_flag = (volatile int*)(sm + S::BAR_OFF + 8 * (2 * S::STAGES));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  pdl_trigger();       // first thing: the successor's prologue overlaps this whole kernel
  if (tid == 0) {
    stamp_start(p.stamp);
    for (int s = 0; s < S::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), NW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  int L = p.L, chunk_keys = p.chunk_keys, n_chunks = p.n_chunks;
  if (p.len_ptr) {   // the length word is written before the forward starts, not by a predecessor kernel
    L = *p.len_ptr;
    attn_chunking(L + p.n, (int)gridDim.x, &chunk_keys, &n_chunks);
  }
  const int n = p.n, hq = p.hq, hkv = p.hkv, qh = p.qh;
  const int chunk = blockIdx.x, grp = blockIdx.y, hk = blockIdx.z;
  if (chunk >= n_chunks) { pdl_wait(); return; }
  const int G = hq / hkv;
  const int head0 = hk * G + grp * qh;                 // first query head of this CTA
  const int heads_here = min(qh, G - grp * qh);
  const int m_valid = heads_here * n;
  const int T = L + n;
  const int key_begin = chunk * chunk_keys;
  const int key_end = min(T, key_begin + chunk_keys);
  const int n_tiles = (key_end - key_begin + AT_KEYS - 1) / AT_KEYS;

  if (warp == NW) {
    // ------------------------------------------------ TMA producer ------------------------------------------------
    if (lane == 0) {
      const uint64_t pol = policy_evict_last();     // the cache is read again by the other head groups and by the next step
      // The host-set test hook (status[1], never written by a kernel): the producer issues nothing and raises the
      // abort flag, so every wait of the compute warps gives up.  Only this thread pays for the read, off the
      // critical path of the others.
      const bool poisoned = p.status && *reinterpret_cast<const volatile int*>(p.status + 1) != 0;
      if (poisoned) *abort_flag = 1;
      bool ok = !poisoned, waited = false;
      uint32_t armed = 0, armed_parity = 0;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int stage = t % S::STAGES;
        const uint32_t phase = (uint32_t)(t / S::STAGES) & 1u;
        const int j0 = key_begin + t * AT_KEYS;
        // rows >= L are written by the predecessor kernel (the block's own K / V)
        if (!waited && j0 + AT_KEYS > L) { pdl_wait(); waited = true; }
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
        mbar_expect_tx(full_bar(stage), S::STAGE_BYTES);
        armed |= 1u << stage;
        armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
        const uint32_t dst = sKV + stage * S::STAGE_BYTES;
        const int row = hk * p.max_seq + j0;
#pragma unroll
        for (int hd = 0; hd < D / 64; ++hd) {
          tma_load_2d(dst + hd * (AT_KEYS * 128), &p.tm_k, full_bar(stage), hd * 64, row, pol);
          tma_load_2d(dst + S::TILE_BYTES + hd * (AT_KEYS * 128), &p.tm_v, full_bar(stage), hd * 64, row, pol);
        }
      }
      if (!waited) pdl_wait();
      if (!ok) {
        if (p.status) atomicCAS(p.status, 0, ST_ATTENTION);
        for (int s = 0; s < S::STAGES; ++s) {      // drain: wait (bounded) for every bulk copy in flight
          if (!(armed & (1u << s))) continue;
          const uint32_t par = (armed_parity >> s) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(s), par) && clock64() - t0 < TC_TIMEOUT) {}
        }
      }
    }
  } else {
    // ------------------------------------------------ compute warps -----------------------------------------------
    // stage Q (rows = heads_here x n; row r -> head r / n, token r % n): written by the predecessor kernel
    const E* q = reinterpret_cast<const E*>(p.q);
    pdl_wait();
    if (tid == 0) stamp_released(p.stamp);
    for (int v = tid; v < ROWS * CH; v += NCT) {
      const int r = v / CH, c = v % CH;
      const bool live = r < m_valid;
      const int hl = live ? r / n : 0, i = live ? r % n : 0;
      cp_async16(sQ + swz_q<D>(r, c), live ? (const void*)(q + ((size_t)i * hq + head0 + hl) * D + c * 8) : (const void*)q, live ? 16 : 0);
    }
    cp_async_commit();
    cp_async_wait<0>();
    asm volatile("bar.sync 1, %0;" ::"n"(NCT) : "memory");

    const int row0 = warp * 16;                       // this warp's rows of the CTA tile
    const bool warp_live = row0 < m_valid;
    const int g = lane >> 2, tq = lane & 3;
    const int r_lo = row0 + g, r_hi = r_lo + 8;       // the two rows this thread owns
    // last visible key (exclusive) of each row
    const int lim_lo = (r_lo < m_valid) ? (p.causal ? L + (r_lo % n) + 1 : T) : 0;
    const int lim_hi = (r_hi < m_valid) ? (p.causal ? L + (r_hi % n) + 1 : T) : 0;
    const float sl2 = rsqrtf((float)D) * LOG2E;       // scores kept in the log2 domain

    uint32_t qf[D / 16][4];
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk)
      ldsm_x4(sQ + swz_q<D>(row0 + (lane & 15), kk * 2 + (lane >> 4)), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
    bool ok = true;

    for (int t = 0; t < n_tiles && ok; ++t) {
      const int stage = t % S::STAGES;
      const uint32_t phase = (uint32_t)(t / S::STAGES) & 1u;
      if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
      const uint32_t kt = sKV + stage * S::STAGE_BYTES;
      const uint32_t vt = kt + S::TILE_BYTES;
      const int j0 = key_begin + t * AT_KEYS;
      if (j0 + AT_KEYS > key_end) {
        // The box reaches past the last key: those V rows hold whatever the cache holds there, and 0 x NaN would
        // poison the P.V product.  Clear them (only ever the last tile of the last chunk, which is never refilled).
        // Every warp clears all of them itself before it reads any: the warps write the same zeros, so no barrier
        // between the warps is needed.
        const int first = key_end - j0;
        for (int v = lane; v < (AT_KEYS - first) * CH; v += 32) {
          const int r = first + v / CH, c = v % CH;
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vt + swz_kv(r, c)), "r"(0u) : "memory");
        }
        __syncwarp();
      }
      if (warp_live) {
        float s[AT_KEYS / 8][4];
#pragma unroll
        for (int i = 0; i < AT_KEYS / 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
          for (int np = 0; np < AT_KEYS / 16; ++np) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(kt + swz_kv(np * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
            mma_16816<E>(s[2 * np], qf[kk], b0, b1);
            mma_16816<E>(s[2 * np + 1], qf[kk], b2, b3);
          }
        }
        // explicit mask among the forward's own rows (keys L .. L+n-1; the words are set up before the chain, not by a
        // kernel of it).  Only the last tile or two hold such keys, so the words are fetched there and kept out of the
        // main loop's registers.
        if (p.row_mask && j0 + AT_KEYS > L) {                // uniform over the warp
          const unsigned long long msk_lo = (r_lo < m_valid) ? p.row_mask[r_lo % n] : 0ull;
          const unsigned long long msk_hi = (r_hi < m_valid) ? p.row_mask[r_hi % n] : 0ull;
#pragma unroll
          for (int nt = 0; nt < AT_KEYS / 8; ++nt) {
            const int j = j0 + nt * 8 + tq * 2;
            if (j >= L && !((msk_lo >> ((j - L) & 63)) & 1ull)) s[nt][0] = -INFINITY;
            if (j + 1 >= L && !((msk_lo >> ((j + 1 - L) & 63)) & 1ull)) s[nt][1] = -INFINITY;
            if (j >= L && !((msk_hi >> ((j - L) & 63)) & 1ull)) s[nt][2] = -INFINITY;
            if (j + 1 >= L && !((msk_hi >> ((j + 1 - L) & 63)) & 1ull)) s[nt][3] = -INFINITY;
          }
        }
        // mask + running max
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
            ldsm_x4_t(vt + swz_kv(kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), dp * 2 + (lane >> 4)), b0, b1, b2, b3);
            mma_16816<E>(o[2 * dp], pa, b0, b1);
            mma_16816<E>(o[2 * dp + 1], pa, b2, b3);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(stage));
    }
    if (!ok && lane == 0 && p.status) atomicCAS(p.status, 0, ST_ATTENTION);

    // ---- partial results: the quad's four lanes hold the row sums in pieces ----
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int r = half ? r_hi : r_lo;
      if (r >= m_valid || !ok) continue;
      const int head = head0 + r / n, i = r % n;
      const size_t slot = ((size_t)head * n + i) * n_chunks + chunk;
      float* dst = p.part_o + slot * D;
#pragma unroll
      for (int dt = 0; dt < D / 8; ++dt) {
        float2 v = half ? make_float2(o[dt][2], o[dt][3]) : make_float2(o[dt][0], o[dt][1]);
        *reinterpret_cast<float2*>(dst + dt * 8 + tq * 2) = v;
      }
      if (tq == 0) p.part_ml[slot] = half ? make_float2(m_hi, l_hi) : make_float2(m_lo, l_lo);
    }
  }
  __syncthreads();     // the producer's copies have all been consumed (or drained) before any thread leaves
  if (tid == 0) stamp_end(p.stamp);
}

// Merge of the key chunks of one (row, head) by one warp: out = sum_c w_c O_c / sum_c w_c l_c, w_c = 2^(m_c - max m).
// Lane j owns D / 32 consecutive output features; the chunk statistics are spread over the lanes.
// The result is stored as `fmt` (XF_*) at element offset out_idx of `out`.
template <int D>
__device__ __forceinline__ void attn_merge_warp(const float* att_o, const float2* att_ml, void* out, size_t out_idx, size_t lo_off,
                                                int fmt, size_t slot0, int n_chunks, int lane, float* amax_out = nullptr) {
  constexpr int VPL = D / 32;
  constexpr int CB = 32;     // chunks whose partial outputs are in flight together
  // The statistics and the first CB partial outputs are requested together: one L2 round trip for up to 32 chunks.
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
  if (amax_out) {     // W8A8: the O projection quantises this row; its maximum as stored (f16) over this head
    float am = 0.f;
#pragma unroll
    for (int i = 0; i < VPL; ++i) am = fmaxf(am, fabsf(__half2float(__ushort_as_half(f16_bits_sat(acc[i] * inv)))));
    am = warp_max(am);
    if (lane == 0) *amax_out = am;
  }
}

// out[i][head] = sum_c w_c O_c / sum_c w_c l_c, w_c = 2^(m_c - max_c m_c): one warp per (row, head), four per CTA
template <int D>
__global__ void __launch_bounds__(128) attn_combine_kernel(const float* __restrict__ part_o, const float2* __restrict__ part_ml,
                                                          void* __restrict__ out, size_t lo_off, int fmt, int n, int hq, int n_chunks,
                                                          const int* __restrict__ len_ptr, int bound, float* __restrict__ amax_out,
                                                          KStamp* stamp) {
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
                       threadIdx.x & 31, amax_out ? amax_out + (size_t)i * hq + head : nullptr);
  }
  __syncthreads();
  if (threadIdx.x == 0) stamp_end(stamp, true);
}

// ---- host side -------------------------------------------------------------------------------------
// The chunk merge that follows either attention kernel.  grid_x: the chunk slots the partials were laid out for.
cudaError_t launch_attn_combine(const float* part_o, const float2* part_ml, const AttnArgs& a, int n_chunks, int grid_x,
                                KStamp* stamp, cudaStream_t st) {
  cudaError_t e;
  if (a.d == 128)
    e = launch_pdl(attn_combine_kernel<128>, dim3((a.n * a.hq + 3) / 4), dim3(128), 0, st, part_o, part_ml, a.out, a.out_lo_off, a.out_fmt,
                   a.n, a.hq, n_chunks, a.len_ptr, grid_x, a.amax_out, stamp);
  else
    e = launch_pdl(attn_combine_kernel<64>, dim3((a.n * a.hq + 3) / 4), dim3(128), 0, st, part_o, part_ml, a.out, a.out_lo_off, a.out_fmt,
                   a.n, a.hq, n_chunks, a.len_ptr, grid_x, a.amax_out, stamp);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// CTAs of 128 rows once the keys make more than this many tiles per 64-row CTA (all SMs busy either way)
constexpr int AT_LONG_KEYS = 3072;

struct AttnPlan { int rows, qh, groups, chunk_keys, n_chunks, bound; };

static int attn_sm_count() {
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
  return v;
}

// rows per CTA: the most query heads of one KV head whose n rows fit
static void attn_rows(int n, int hq, int hkv, int rows_cap, int* qh, int* groups) {
  const int G = hq / hkv;
  *qh = 1;
  for (int c = G; c >= 1; --c)
    if (c * n <= rows_cap) { *qh = c; break; }
  *groups = ceil_div(G, *qh);
}

static AttnPlan attn_plan(int n, int T, int hq, int hkv, bool long_cache) {
  AttnPlan p;
  p.rows = (long_cache && (hq / hkv) * n > 64) ? 128 : 64;
  attn_rows(n, hq, hkv, p.rows, &p.qh, &p.groups);
  // 64-row CTAs sit two to an SM, 128-row CTAs one
  p.bound = ceil_div((p.rows == 64 ? 2 : 1) * attn_sm_count(), hkv * p.groups);
  attn_chunking(T, p.bound, &p.chunk_keys, &p.n_chunks);
  return p;
}

size_t attention_mma_workspace_bytes(int n, int hq, int hkv, int d) {
  size_t worst = 0;
  for (int m = 1; m <= n; ++m) {
    const int row_caps[2] = {64, 128};
    for (int rows : row_caps) {
      int qh, groups;
      attn_rows(m, hq, hkv, rows, &qh, &groups);
      const size_t slots = (size_t)hq * m * ceil_div(2 * 148, hkv * groups);
      if (slots > worst) worst = slots;
    }
  }
  return worst * ((size_t)d * 4 + 8) + 256;
}

template <int D, typename E, int ROWS>
static cudaError_t attn_launch_t(const AttnArgs& a, const AttnPlan& pl, cudaStream_t st) {
  using S = AtSmem<D, ROWS>;
  // with the length on the device the grid is sized for the most chunks any length can give
  int grid_x = pl.n_chunks;
  if (a.len_ptr) { grid_x = pl.bound; const int tmax = ceil_div(a.max_seq, AT_KEYS); if (grid_x > tmax) grid_x = tmax; }
  const size_t slots = (size_t)a.hq * a.n * grid_x;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  const int kind = a.kv_type == KV_F16 ? TM_F16 : TM_BF16;
  if (!make_tmap(&p.tm_k, a.kc, a.hkv * a.max_seq, D, AT_KEYS, kind) || !make_tmap(&p.tm_v, a.vc, a.hkv * a.max_seq, D, AT_KEYS, kind))
    return cudaErrorInvalidValue;
  p.q = a.q;
  p.part_o = (float*)a.workspace;
  p.part_ml = (float2*)((char*)a.workspace + ((slots * D * 4 + 255) / 256) * 256);
  p.n = a.n; p.L = a.cache_len; p.max_seq = a.max_seq; p.hq = a.hq; p.hkv = a.hkv; p.qh = pl.qh;
  p.chunk_keys = pl.chunk_keys; p.n_chunks = pl.n_chunks; p.causal = a.row_mask ? 0 : a.causal; p.row_mask = a.row_mask; p.len_ptr = a.len_ptr; p.status = a.status; p.stamp = a.stamp;
  static bool attr_set[MAX_DEVICES] = {};
  cudaError_t e = ensure_dynamic_smem(attn_mma_kernel<D, E, ROWS>, S::TOTAL, attr_set);
  if (e != cudaSuccess) return e;
  dim3 grid(grid_x, pl.groups, a.hkv);
  e = launch_pdl(attn_mma_kernel<D, E, ROWS>, grid, dim3(S::THREADS), (size_t)S::TOTAL, st, p);
  if (e != cudaSuccess) return e;
  return launch_attn_combine(p.part_o, p.part_ml, a, pl.n_chunks, grid_x, a.stamp ? a.stamp + 1 : nullptr, st);
}

template <int D, typename E>
static cudaError_t attn_launch_r(const AttnArgs& a, const AttnPlan& pl, cudaStream_t st) {
  return pl.rows == 128 ? attn_launch_t<D, E, 128>(a, pl, st) : attn_launch_t<D, E, 64>(a, pl, st);
}

bool attention_long_cache(int keys) { return keys > AT_LONG_KEYS; }

int launch_attention_mma(const AttnArgs& a, cudaStream_t st, cudaError_t* err) {
  const bool long_cache = a.long_cache >= 0 ? a.long_cache != 0 : attention_long_cache(a.cache_len + a.n);
  if (!a.workspace) { *err = cudaErrorInvalidValue; return -1; }
  const AttnPlan pl = attn_plan(a.n, a.cache_len + a.n, a.hq, a.hkv, long_cache);
  if (a.kv_type == KV_F16) *err = (a.d == 128) ? attn_launch_r<128, __half>(a, pl, st) : attn_launch_r<64, __half>(a, pl, st);
  else *err = (a.d == 128) ? attn_launch_r<128, bf16>(a, pl, st) : attn_launch_r<64, bf16>(a, pl, st);
  return *err == cudaSuccess ? 2 : -1;
}

}  // namespace fdk
