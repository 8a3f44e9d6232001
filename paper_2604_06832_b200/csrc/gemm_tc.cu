// Small-M weight-streaming GEMM for sm_100a: y[m, n] = sum_k x[m, k] w[n, k], m <= 64.
//
// The weight matrix is the MMA "A" operand (128 output features per tile fill the tensor-core M
// dimension), the m activation rows are the MMA "N" dimension (padded to 16/32/48/64), so a CTA
// streams 128 x K weights once while the tiny activation tile comes from L2.  Weights and
// activations are staged by TMA (128-byte swizzle, K-major) into a ring of shared-memory stages;
// one elected thread issues tcgen05.mma with fp32 accumulators in tensor memory (two accumulator
// buffers, so the epilogue of one work item overlaps the mainloop of the next); four epilogue warps
// read the accumulators with tcgen05.ld.  CTAs are persistent over a static round-robin list of
// work items (tile, K-split).  bf16 weights: the activations arrive as two bf16 planes, hi = bf16(v) and
// lo = bf16(v - hi); both land side by side in the stage and form ONE MMA operand of twice the rows, so every streamed
// weight tile is read from shared memory once and multiplied by both; the epilogue adds the two halves of the
// accumulator.  The activation side of the product thus carries ~16 significant bits at no extra HBM traffic.  FP8-E4M3 weights take the
// same road with half the bytes: the byte tile lands in the stage, four converter warps widen it exactly to f16
// (one cvt per pair) into a swizzled buffer of its own, and the MMA (f16 x f16, activations stored as f16) reads
// that buffer; the per-channel scales are applied by the epilogues.
// Every mbarrier wait is bounded: on a timeout the CTA records an
// error code in a status word, drains its own bulk copies, frees its tensor memory and returns.
#include <cuda.h>

#include <map>
#include <mutex>
#include <tuple>

#include "kernels.h"
#include "tc_ptx.cuh"

namespace fdk {

constexpr int TC_THREADS = 192;       // warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 epilogue
constexpr int TC_THREADS_FP8 = 320;   // + warps 6..9: e4m3 -> bf16 converters
constexpr int TC_A_BYTES = TC_BM * TC_BK * 2;   // a bf16 weight tile
constexpr int TC_NCONV = 2;           // converted-tile buffers (fp8 only)

enum { TC_ERR_PRODUCER = ST_PRODUCER, TC_ERR_MMA = ST_MMA, TC_ERR_EPILOGUE = ST_EPILOGUE };

struct TcParams {
  CUtensorMap tm_w[3];  // weight matrices, box {64 k, 64 rows}
  CUtensorMap tm_x;     // activations (hi plane, or the only one), box {64 k, m_pad rows}
  CUtensorMap tm_xl;    // lo plane of the activations (has_lo)
  int has_lo;
  int n_out[3];         // rows (output features) of each matrix
  int tile_begin[4];    // first tile of each matrix; [n_mats] = total tiles
  int out_col[3];       // column of each matrix's first feature in the output row
  const float* scale[3];
  const float* bias[3];
  int n_mats, kblocks, splits, kb_per_split, m, mode;
  float* part;          // [splits][m][ldp]     (PARTIAL)
  int ldp;
  float* y;             // [m][ldy]             (DIRECT)
  int ldy, accumulate;
  void* act;            // [m][inter]           (SWIGLU), stored as act_fmt (XF_*), lo plane act_lo_off elements on
  size_t act_lo_off;
  int act_fmt, inter;
  // RMSNorm folded into the consumer: x holds bf16(h * gain); the per-row factor rsqrt(mean(h^2) + eps)
  // is applied to the accumulators.  ssq_in[row][nt_in] holds partial sums of h^2 (null: factor 1).
  const float* ssq_in;
  int nt_in;
  float inv_h, eps;
  // LOGITS mode: per (tile, lane quarter, row) softmax statistics of the 32 columns a warp holds, the
  // mask token's column excluded: (max, sum exp(l - max), argmax column)
  float4* stats;        // [tiles * 4][m]
  int mask_id, write_logits;
  int* status;          // device words: [0] set non-zero when a wait timed out; [1] read at start: non-zero makes
                        // every role take its give-up path at once (a host-set test hook for that path)
  KStamp* stamp;        // in-chain timing of this launch (null: off)
  // TC_KIND_A8: amax_in[row][n_amax_in] = partial maxima of |x[row]| left by the producer of x; the row's quantisation
  // scale is their maximum / 448.  SWIGLU mode also raises amax_out[row] (atomic maximum; zero before the launch) to
  // the maximum of |act[row]| as stored, for the consumer of `act`.
  const float* amax_in; int n_amax_in;
  float* amax_out;
};

// Operand kinds of the kernel:
//   TC_KIND_BF16: bf16 weights x bf16 hi/lo activation planes
//   TC_KIND_FP8 : e4m3 weights widened to f16 by converter warps x f16 activations
//   TC_KIND_A8  : e4m3 weights x activations quantised to e4m3 per row inside the kernel (W8A8, Sec. 3.4 "System
//                 integration"); a k-block is 128 elements, the byte tile of the weights is the MMA operand as it lands
enum { TC_KIND_BF16 = 0, TC_KIND_FP8 = 1, TC_KIND_A8 = 2 };

template <int M_PAD, int KIND>
struct TcSmem {
  static constexpr bool FP8 = KIND == TC_KIND_FP8, A8 = KIND == TC_KIND_A8;
  static constexpr int STAGES = FP8 ? 6 : (M_PAD <= 32 ? 4 : 3);       // two CTAs per SM must fit (A8, M_PAD > 32: one)
  static constexpr int KB_ELEMS = A8 ? 2 * TC_BK : TC_BK;              // k per stage
  static constexpr int W_BYTES = FP8 ? TC_BM * TC_BK : TC_A_BYTES;     // weight tile as it is streamed
  static constexpr int B_BYTES = M_PAD * TC_BK * 2;                    // one activation plane (A8: one 64-k half, f16)
  static constexpr int X_PLANES = FP8 ? 1 : 2;                         // f16; bf16 hi + lo; A8: two 64-k halves
  static constexpr int STAGE_BYTES = W_BYTES + X_PLANES * B_BYTES;
  static constexpr int CONV_OFF = STAGES * STAGE_BYTES;                // tiles made by the converters
  static constexpr int CONV_BYTES = FP8 ? TC_A_BYTES : (A8 ? M_PAD * 128 : 0);   // f16 weight tile / e4m3 activation tile
  static constexpr int EX_OFF = CONV_OFF + TC_NCONV * CONV_BYTES;      // SwiGLU epilogue: gate/up exchange
  static constexpr int EX_ROWS = KIND != TC_KIND_BF16 ? 16 : 32;       // rows that pass through it per round
  static constexpr int EX_ROUNDS = (M_PAD + EX_ROWS - 1) / EX_ROWS;
  static constexpr int EX_BYTES = (M_PAD / EX_ROUNDS) * 256;
  static constexpr int BAR_OFF = EX_OFF + EX_BYTES;
  static constexpr int ROWSC_OFF = BAR_OFF + 256;                      // A8: the rows' quantisation scales and their reciprocals
  static constexpr int TOTAL = ROWSC_OFF + 512 + 1024;  // + alignment slack
};

// sixteen e4m3 bytes -> sixteen f16 (exact: every e4m3 value, subnormals included, is an f16 value)
__device__ __forceinline__ void e4m3x16_to_f16(const uint4& in, uint4& lo, uint4& hi) {
  const uint32_t w[4] = {in.x, in.y, in.z, in.w};
  uint32_t o[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int hsel = 0; hsel < 2; ++hsel) {
      const unsigned short two = (unsigned short)(hsel ? (w[i] >> 16) : (w[i] & 0xffffu));
      asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(o[2 * i + hsel]) : "h"(two));
    }
  }
  lo = make_uint4(o[0], o[1], o[2], o[3]);
  hi = make_uint4(o[4], o[5], o[6], o[7]);
}

// Widen NP 16-byte pieces (tid, tid + stride, ...) of an 8 KB e4m3 tile (rows of 64 bytes) into the 128-byte-swizzled
// f16 tile the MMA descriptor expects.
template <int NP>
__device__ __forceinline__ void convert_pieces(const uint8_t* src, uint32_t dst, int tid, int stride) {
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int piece = tid + stride * i, r = piece >> 2, c = piece & 3;     // row, 16-byte piece of the row
    const uint4 in = *reinterpret_cast<const uint4*>(src + piece * 16);
    uint4 lo, hi;
    e4m3x16_to_f16(in, lo, hi);
    const uint32_t row = dst + r * 128;
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (((2 * c) ^ (r & 7)) << 4)), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (((2 * c + 1) ^ (r & 7)) << 4)), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
  }
}

// Quantise NP 16-byte pieces (tid, tid + stride, ...) of the activation tile of one stage -- two 128-byte-swizzled f16
// halves of 64 k each -- into the 128-byte-swizzled e4m3 tile [M_PAD rows][128 k] the MMA reads: code = e4m3(x / scale
// of the row), float32 quotient, round to nearest even, saturating.  The quotient is formed without the division
// routine: with y = RN(1 / scale), q0 = RN(x y) and the exact remainder r = x - q0 scale (one FMA), RN(q0 + r y) is the
// correctly rounded x / scale (Markstein's correction step; no operand here is zero, infinite or subnormal except
// x = 0, which gives 0 either way).
template <int M_PAD, int NP>
__device__ __forceinline__ void quantize_pieces(const uint8_t* x_tile, uint32_t dst, const volatile float2* row_scale, int tid, int stride) {
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    const int piece = tid + stride * i;
    if (piece >= M_PAD * 8) break;
    const int r = piece >> 3, j = piece & 7;                 // row, 16-byte piece (16 k) of the output row
    const uint8_t* half = x_tile + (j >> 2) * (M_PAD * 128) + r * 128;
    const int c0 = 2 * (j & 3);
    const uint4 a = *reinterpret_cast<const uint4*>(half + ((c0 ^ (r & 7)) << 4));
    const uint4 b = *reinterpret_cast<const uint4*>(half + (((c0 + 1) ^ (r & 7)) << 4));
    const float sc = row_scale[r].x, rinv = row_scale[r].y;
    const uint32_t in[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t out[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      unsigned short pair[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const __half2 hv = *reinterpret_cast<const __half2*>(&in[2 * w + h]);
        const float a0 = __low2float(hv), a1 = __high2float(hv);
        const float q0 = a0 * rinv, q1 = a1 * rinv;
        const float x0 = fmaf(fmaf(-q0, sc, a0), rinv, q0), x1 = fmaf(fmaf(-q1, sc, a1), rinv, q1);
        asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair[h]) : "f"(x1), "f"(x0));   // first source -> upper byte
      }
      out[w] = (uint32_t)pair[0] | ((uint32_t)pair[1] << 16);
    }
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + r * 128 + ((j ^ (r & 7)) << 4)), "r"(out[0]), "r"(out[1]), "r"(out[2]), "r"(out[3]) : "memory");
  }
}

template <int M_PAD, int KIND>
__global__ void __launch_bounds__(KIND != TC_KIND_BF16 ? TC_THREADS_FP8 : TC_THREADS, 1) gemm_tc_kernel(const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  using L = TcSmem<M_PAD, KIND>;
  constexpr bool A8 = KIND == TC_KIND_A8;
  constexpr bool FP8 = KIND != TC_KIND_BF16;       // a converter stage sits between the ring and the MMA
  constexpr bool WIDEN = KIND == TC_KIND_FP8;      // ... which widens the weight tile (A8: quantises the activation tile)
  constexpr int TC_STAGES = L::STAGES;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t bar0 = base + L::BAR_OFF;
  // barrier slots (8 bytes each): full[S], empty[S], tmem_full[2], tmem_empty[2], conv_full[2], conv_empty[2]
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (TC_STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * TC_STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * TC_STAGES + 2 + a); };
  auto cfull_bar = [&](int c) { return bar0 + 8u * (2 * TC_STAGES + 4 + c); };
  auto cempty_bar = [&](int c) { return bar0 + 8u * (2 * TC_STAGES + 6 + c); };
  // SwiGLU epilogue, per warp pair pr: exchange buffer written (exw) / read (exr), two arrivals each
  auto exw_bar = [&](int pr) { return bar0 + 8u * (2 * TC_STAGES + 10 + pr); };
  auto exr_bar = [&](int pr) { return bar0 + 8u * (2 * TC_STAGES + 12 + pr); };
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(sm + L::BAR_OFF + 8 * (2 * TC_STAGES + 8));
  volatile int* abort_flag = (volatile int*)(sm + L::BAR_OFF + 8 * (2 * TC_STAGES + 8) + 8);
  volatile float2* row_scale = reinterpret_cast<volatile float2*>(sm + L::ROWSC_OFF);   // A8 only: (scale, RN(1 / scale))

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // two accumulator buffers; bf16 weights: each holds the hi-plane product in columns [0, M_PAD) and the lo-plane
  // product in [M_PAD, 2 M_PAD)
  constexpr int ACC_COLS = FP8 ? M_PAD : 2 * M_PAD;
  constexpr int TMEM_COLS = (2 * ACC_COLS <= 32) ? 32 : ((2 * ACC_COLS <= 64) ? 64 : ((2 * ACC_COLS <= 128) ? 128 : 256));

  // fp8 launches in which no CTA has a second work item: the epilogue warps, idle until the accumulator is complete,
  // widen half of every weight tile beside the four converter warps
  const bool helpers = WIDEN && p.tile_begin[p.n_mats] * p.splits <= (int)gridDim.x;
  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
    for (int c = 0; c < TC_NCONV; ++c) { mbar_init(cfull_bar(c), helpers ? 8 : 4); mbar_init(cempty_bar(c), 1); }
    for (int pr = 0; pr < 2; ++pr) { mbar_init(exw_bar(pr), 2); mbar_init(exr_bar(pr), 2); }
    stamp_start(p.stamp);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Dependents may start only now that this CTA holds its tensor memory: a successor CTA that allocated first and then
  // waited for this grid could otherwise keep it from ever getting any.
  pdl_trigger();

  const int total_tiles = p.tile_begin[p.n_mats];
  const int n_items = total_tiles * p.splits;

  const int kbps = p.kb_per_split, kblocks = p.kblocks;
  auto convert_all = [&](int cvt_tid) -> bool {
    int stage = 0, cbuf = 0;
    uint32_t phase = 0, cphase = 0;
    for (int it = blockIdx.x; it < n_items; it += gridDim.x) {
      const int split = it / total_tiles;
      const int kb0 = split * kbps;
      const int kb1 = min(kblocks, kb0 + kbps);
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag) || !mbar_wait(cempty_bar(cbuf), cphase ^ 1u, abort_flag)) return false;
        const uint8_t* src = sm + stage * L::STAGE_BYTES;
        const uint32_t dst = base + L::CONV_OFF + cbuf * L::CONV_BYTES;
        if (A8) quantize_pieces<M_PAD, (M_PAD * 8 + 127) / 128>(src + L::W_BYTES, dst, row_scale, cvt_tid, 128);
        else if (helpers) convert_pieces<2>(src, dst, cvt_tid, 256);
        else convert_pieces<4>(src, dst, cvt_tid, 128);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> the MMA's async-proxy reads
        __syncwarp();
        if (lane == 0) mbar_arrive(cfull_bar(cbuf));
        if (++cbuf == TC_NCONV) { cbuf = 0; cphase ^= 1u; }
        if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
      }
    }
    return true;
  };

  if (warp == 0) {
    // ------------------------------------------------ TMA producer ------------------------------------------------
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
      // The host-set test hook (status[1]; written by the host only, never by a kernel of the chain, so it may be read
      // before the wait): the producer issues nothing and raises the abort flag, which every other role's first wait
      // sees -- all leave by the path a timed-out wait takes.  Only this thread pays for the read.
      const bool poisoned = p.status && *reinterpret_cast<const volatile int*>(p.status + 1) != 0;
      if (poisoned) *abort_flag = 1;
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0;           // bit s: full[s] armed and not yet known complete
      uint32_t armed_parity = 0;    // bit s: parity of that arming
      bool ok = !poisoned;
      bool waited = false;
      int n_pend = 0, pend_stage[TC_STAGES], pend_kb[TC_STAGES];
      const uint32_t stage_tx = L::W_BYTES + ((A8 || p.has_lo) ? 2 : 1) * L::B_BYTES;
      auto load_x = [&](int st_, int kb_) {
        const uint32_t dst = base + st_ * L::STAGE_BYTES + L::W_BYTES;
        tma_load_2d(dst, &p.tm_x, full_bar(st_), kb_ * L::KB_ELEMS, 0, pol_x);
        if (A8) tma_load_2d(dst + L::B_BYTES, &p.tm_x, full_bar(st_), kb_ * L::KB_ELEMS + TC_BK, 0, pol_x);   // second 64 k
        if (!FP8 && p.has_lo) tma_load_2d(dst + L::B_BYTES, &p.tm_xl, full_bar(st_), kb_ * TC_BK, 0, pol_x);
      };
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        const int tile = it % total_tiles, split = it / total_tiles;
        int mi = 0, r0 = 0;
        if (p.mode != TC_MODE_SWIGLU) {
          while (mi + 1 < p.n_mats && tile >= p.tile_begin[mi + 1]) ++mi;
          r0 = (tile - p.tile_begin[mi]) * TC_BM;
        }
        const int kb0 = split * p.kb_per_split;
        const int kb1 = min(p.kblocks, kb0 + p.kb_per_split);
        // Every CTA walks its k-blocks from a different starting point (and wraps): the activation tile of a k-block
        // is the same few L2 lines for all CTAs, and in lockstep they would all ask for them at the same moment.
        const int nkb = kb1 - kb0;
        const int rot = (int)((blockIdx.x * 7u) % (unsigned)nkb);
        for (int j = 0; j < nkb; ++j) {
          const int kb = kb0 + ((j + rot) >= nkb ? j + rot - nkb : j + rot);
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t a_dst = base + stage * L::STAGE_BYTES;
          mbar_expect_tx(full_bar(stage), stage_tx);
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (p.mode == TC_MODE_SWIGLU) {
            // 64 features per tile: their gate rows fill TMEM lanes 0..63, their up rows lanes 64..127
            tma_load_2d(a_dst, &p.tm_w[0], full_bar(stage), kb * L::KB_ELEMS, tile * 64, pol_w);
            tma_load_2d(a_dst + L::W_BYTES / 2, &p.tm_w[1], full_bar(stage), kb * L::KB_ELEMS, tile * 64, pol_w);
          } else {
            tma_load_2d(a_dst, &p.tm_w[mi], full_bar(stage), kb * L::KB_ELEMS, r0, pol_w);
            tma_load_2d(a_dst + L::W_BYTES / 2, &p.tm_w[mi], full_bar(stage), kb * L::KB_ELEMS, r0 + 64, pol_w);
          }
          // The weights do not depend on the predecessor kernel: the first ring of weight loads is issued before waiting
          // for it; the activation tiles of those stages follow once it has completed.
          if (waited) {
            load_x(stage, kb);
          } else {
            pend_stage[n_pend] = stage; pend_kb[n_pend] = kb;
            if (++n_pend == TC_STAGES) {
              pdl_wait();
              stamp_released(p.stamp);
              waited = true;
              for (int j = 0; j < n_pend; ++j) load_x(pend_stage[j], pend_kb[j]);
            }
          }
          if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!waited) {
        pdl_wait();
        stamp_released(p.stamp);
        for (int j = 0; j < n_pend; ++j) load_x(pend_stage[j], pend_kb[j]);
      }
      if (!ok) {
        atomicCAS(p.status, 0, TC_ERR_PRODUCER);
        // drain: wait (bounded) for every bulk copy this thread has in flight
        for (int s = 0; s < TC_STAGES; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t par = (armed_parity >> s) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(s), par) && clock64() - t0 < TC_TIMEOUT) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer --------------------------------------------------
    if (lane == 0) {
      const bool two_planes = !FP8 && p.has_lo;
      const uint32_t idesc = A8 ? umma_idesc_e4m3(M_PAD) : (FP8 ? umma_idesc_f16(M_PAD) : umma_idesc_bf16(two_planes ? 2 * M_PAD : M_PAD));
      int stage = 0, cbuf = 0;
      uint32_t phase = 0, cphase = 0;
      int local = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++local) {
        const int split = it / total_tiles;
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
        const int kb0 = split * p.kb_per_split;
        const int kb1 = min(p.kblocks, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; ++kb) {
          // fp8: the converters have waited for the stage and left their tile in buffer cbuf (the widened weights; A8:
          // the quantised activations, the weight bytes being read from the stage itself, whose barrier this thread
          // then observes too)
          if (!mbar_wait(FP8 ? cfull_bar(cbuf) : full_bar(stage), FP8 ? cphase : phase, abort_flag)) { ok = false; break; }
          if (A8 && !mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = base + stage * L::STAGE_BYTES;
          const uint32_t c_addr = base + L::CONV_OFF + cbuf * L::CONV_BYTES;
          const uint64_t adesc = umma_desc_sw128(WIDEN ? c_addr : a_addr);
          const uint64_t bdesc = umma_desc_sw128(A8 ? c_addr : a_addr + L::W_BYTES);
          if (A8) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)      // 32 bytes of k per instruction
              umma_f8(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
          } else {
#pragma unroll
            for (int kk = 0; kk < TC_BK / 16; ++kk)
              umma_bf16(d_tmem, adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));
          if (FP8) {
            umma_commit(cempty_bar(cbuf));
            if (++cbuf == TC_NCONV) { cbuf = 0; cphase ^= 1u; }
          }
          if (++stage == TC_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(tfull_bar(acc));
      }
      if (!ok) atomicCAS(p.status, 0, TC_ERR_MMA);
    }
  } else if (FP8 && warp >= 6) {
    // ------------------------------------------------ converters -----------------------------------------------------
    // TC_KIND_FP8: 128 threads (256 with the epilogue warps helping): thread t widens the 16-byte pieces t, t + 128
    // (256), ... of each 8 KB byte tile.  TC_KIND_A8: the same threads quantise the activation tile; first they form
    // every row's scale = max of the producer's partial maxima / 448 (two threads per row; 1 for an all-zero row).
    if (A8) {
      const int t = (int)threadIdx.x - 192, r = t >> 1;
      pdl_wait();                      // the partial maxima are the predecessor's
      float mx = 0.f;
      if (r < p.m && p.amax_in) {
        // sixteen loads in flight per thread: the usual counts (a few dozen partial maxima) cost one round trip
        const float* src = p.amax_in + (size_t)r * p.n_amax_in;
        for (int i0 = (t & 1); i0 < p.n_amax_in; i0 += 32) {
          float v[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) v[u] = (i0 + 2 * u < p.n_amax_in) ? __ldcg(src + i0 + 2 * u) : 0.f;
#pragma unroll
          for (int u = 0; u < 16; ++u) mx = fmaxf(mx, v[u]);
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      if ((t & 1) == 0) {
        const float sc = mx > 0.f ? __fdiv_rn(mx, 448.f) : 1.f;
        row_scale[r].x = sc;
        row_scale[r].y = __frcp_rn(sc);
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");
    }
    if (!convert_all(threadIdx.x - 192) && threadIdx.x == 192) atomicCAS(p.status, 0, TC_ERR_MMA);
  } else {
    // ------------------------------------------------ epilogue warps ----------------------------------------------
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    int local = 0;
    bool ok = true;
    if (helpers) ok = convert_all(128 + (int)threadIdx.x - 64);
    pdl_wait();   // the epilogue reads the predecessor's row statistics and overwrites buffers it may still be reading
    // folded RMSNorm: lane l keeps the factor of rows l and l + 32; broadcast by shuffle where needed
    float rs0 = 1.f, rs1 = 1.f;
    if (p.ssq_in) {
      if (lane < p.m) {
        float s = 0.f;
        for (int t = 0; t < p.nt_in; ++t) s += p.ssq_in[(size_t)lane * p.nt_in + t];
        rs0 = rsqrtf(s * p.inv_h + p.eps);
      }
      if (lane + 32 < p.m) {
        float s = 0.f;
        for (int t = 0; t < p.nt_in; ++t) s += p.ssq_in[(size_t)(lane + 32) * p.nt_in + t];
        rs1 = rsqrtf(s * p.inv_h + p.eps);
      }
    }
    for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++local) {
      const int tile = it % total_tiles, split = it / total_tiles;
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (A8 && local == 0) {
        // the converters left every row's quantisation scale in shared memory before the first tile they made; the
        // accumulator holds sums of code products, so the scale multiplies the folded norm factor
        rs0 *= row_scale[lane].x;
        rs1 *= row_scale[lane + 32].x;
      }
      float v[M_PAD];
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * ACC_COLS);
#pragma unroll
      for (int c = 0; c < M_PAD; c += 16) tmem_ld16(taddr + c, v + c);
      if (!FP8 && p.has_lo) {      // the low-order plane's product sits M_PAD columns further on
#pragma unroll
        for (int c = 0; c < M_PAD; c += 16) {
          float lo[16];
          tmem_ld16(taddr + M_PAD + c, lo);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int i = 0; i < 16; ++i) v[c + i] += lo[i];
        }
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));

      if (p.mode == TC_MODE_SWIGLU) {
        // Warps 0, 1 of the epilogue hold the gate values of features 32 pr + lane, warps 2, 3 the up values of the
        // same features.  Each warp of a pair finishes half of the rows: it hands the other half of its values
        // (scaled) to its partner through shared memory and takes the partner's values for its own rows.
        constexpr int HALF = M_PAD / 2;
        constexpr int ROUNDS = L::EX_ROUNDS;
        static_assert(HALF % ROUNDS == 0, "rows per round");
        constexpr int HR = HALF / ROUNDS;
        const int side = q >> 1, pr = q & 1;
        const int col = tile * 64 + pr * 32 + lane;
        const bool live = col < p.inter;
        const float sc = (live && p.scale[side]) ? p.scale[side][col] : 1.f;
        float* ex = reinterpret_cast<float*>(sm + L::EX_OFF) + pr * (2 * HR * 32);   // [side][HR rows][32 lanes]
#pragma unroll
        for (int r = 0; r < ROUNDS; ++r) {
          const uint32_t par = (uint32_t)(local * ROUNDS + r) & 1u;
#pragma unroll
          for (int b = 0; b < HR; ++b) {
            // the gate side finishes rows 0 .. HALF-1 and sends its values of rows HALF ..; the up side the reverse
            const int lo = r * HR + b, hi = HALF + r * HR + b;
            const float rs_lo = __shfl_sync(0xffffffffu, (lo < 32) ? rs0 : rs1, lo & 31);
            const float rs_hi = __shfl_sync(0xffffffffu, (hi < 32) ? rs0 : rs1, hi & 31);
            ex[(side * HR + b) * 32 + lane] = side ? v[lo] * sc * rs_lo : v[hi] * sc * rs_hi;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(exw_bar(pr));
          if (!mbar_wait(exw_bar(pr), par, abort_flag)) { ok = false; break; }
#pragma unroll
          for (int b = 0; b < HR; ++b) {
            const int lo = r * HR + b, hi = HALF + r * HR + b;
            const float rs_lo = __shfl_sync(0xffffffffu, (lo < 32) ? rs0 : rs1, lo & 31);
            const float rs_hi = __shfl_sync(0xffffffffu, (hi < 32) ? rs0 : rs1, hi & 31);
            const float other = ex[((1 - side) * HR + b) * 32 + lane];
            const float mine = side ? v[hi] * sc * rs_hi : v[lo] * sc * rs_lo;
            const float g = side ? other : mine, u = side ? mine : other;
            const int row = side ? hi : lo;
            const float val = g / (1.f + __expf(-g)) * u;
            if (live && row < p.m) store_act(p.act, p.act_lo_off, (size_t)row * p.inter + col, val, p.act_fmt);
            if (A8 && p.amax_out) {
              // maximum of |act| as stored (f16) over this warp's 32 features, for the consumer's quantiser; values
              // are non-negative, so their bit patterns order like integers (and the result does not depend on order)
              float am = (live && row < p.m) ? fabsf(__half2float(__ushort_as_half(f16_bits_sat(val)))) : 0.f;
              am = warp_max(am);
              if (lane == 0 && row < p.m && am > 0.f) atomicMax(reinterpret_cast<int*>(p.amax_out) + row, __float_as_int(am));
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(exr_bar(pr));
          // the buffer may be rewritten once the partner has read it too
          if (!mbar_wait(exr_bar(pr), par, abort_flag)) { ok = false; break; }
        }
        if (!ok) break;
      } else if (p.mode == TC_MODE_LOGITS) {
        const int n = tile * TC_BM + q * 32 + lane;          // vocabulary id held by this lane
        const bool in_range = n < p.n_out[0];
        const bool counted = in_range && n != p.mask_id;
        const float sc = (in_range && p.scale[0]) ? p.scale[0][n] : 1.f;
#pragma unroll
        for (int b = 0; b < M_PAD; ++b) {
          if (b >= p.m) break;                                // uniform across the warp
          const float rs = __shfl_sync(0xffffffffu, (b < 32) ? rs0 : rs1, b & 31);
          const float l = v[b] * sc * rs;
          if (p.write_logits && in_range) p.y[(size_t)b * p.ldy + n] = l;
          float mx = counted ? l : -INFINITY;
          int ix = counted ? n : 0x7fffffff;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float omx = __shfl_xor_sync(0xffffffffu, mx, o);
            const int oix = __shfl_xor_sync(0xffffffffu, ix, o);
            if (omx > mx || (omx == mx && oix < ix)) { mx = omx; ix = oix; }
          }
          float e = (counted && mx > -INFINITY) ? __expf(l - mx) : 0.f;
          e = warp_sum(e);
          if (lane == 0) p.stats[(size_t)(tile * 4 + q) * p.m + b] = make_float4(mx, e, __int_as_float(ix), 0.f);
        }
      } else {
        int mi = 0;
        while (mi + 1 < p.n_mats && tile >= p.tile_begin[mi + 1]) ++mi;
        const int n = (tile - p.tile_begin[mi]) * TC_BM + q * 32 + lane;
        const bool in_range = n < p.n_out[mi];
        const int col = p.out_col[mi] + n;
        if (p.mode == TC_MODE_PARTIAL) {
          if (in_range) {
            float* dst = p.part + (size_t)split * p.m * p.ldp + col;
#pragma unroll
            for (int b = 0; b < M_PAD; ++b)
              if (b < p.m) dst[(size_t)b * p.ldp] = v[b];
          }
        } else {
          const float sc = (in_range && p.scale[mi]) ? p.scale[mi][n] : 1.f;
          const float bi = (in_range && p.bias[mi]) ? p.bias[mi][n] : 0.f;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) {
            const float rs = __shfl_sync(0xffffffffu, (b < 32) ? rs0 : rs1, b & 31);
            if (in_range && b < p.m) {
              float* dst = p.y + (size_t)b * p.ldy + col;
              float r = v[b] * sc * rs + bi;
              if (p.accumulate) r += *dst;
              *dst = r;
            }
          }
        }
      }
    }
    if (!ok && lane == 0) atomicCAS(p.status, 0, TC_ERR_EPILOGUE);
  }

  // ---- teardown: every thread arrives here, whatever happened ----
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (threadIdx.x == 0) stamp_end(p.stamp);
}

// ================================================================================================
// host side
// ================================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  });
  return fn;
}

// 2-D row-major [rows, cols] tensor, box {64 columns, box_rows}, zero OOB fill.  16-bit elements (TM_BF16, TM_F16):
// 128-byte swizzle (rows of the box are 128 bytes); e4m3 bytes: TM_E4M3 no swizzle (rows of 64 bytes, widened by the
// converter warps), TM_E4M3_128 a box of 128 columns with the 128-byte swizzle (the tile is an MMA operand as it lands).
bool make_tmap(CUtensorMap* tm, const void* ptr, int rows, int cols, int box_rows, int kind) {
  typedef std::tuple<const void*, int, int, int, int> Key;
  static std::map<Key, CUtensorMap> cache;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  const bool fp8 = kind == TM_E4M3 || kind == TM_E4M3_128;
  const bool wide = kind == TM_E4M3_128;
  Key key(ptr, rows, cols, box_rows, kind);
  auto it = cache.find(key);
  if (it != cache.end()) { *tm = it->second; return true; }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * (fp8 ? 1 : 2)};
  cuuint32_t box[2] = {(cuuint32_t)(wide ? 2 * TC_BK : TC_BK), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapDataType dt = fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : (kind == TM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16);
  CUresult r = fn(tm, dt, 2, const_cast<void*>(ptr), dims, strides,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, (fp8 && !wide) ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *tm;
  return true;
}

// SM count of the current device (cached per device: one process may drive several GPUs)
static int sm_count() {
  static int n[MAX_DEVICES] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 148;
  if (!n[dev]) {
    int v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    n[dev] = v > 0 ? v : 148;
  }
  return n[dev];
}

static int pad_m(int m) { return m <= 16 ? 16 : (m <= 32 ? 32 : (m <= 48 ? 48 : 64)); }

// Split-K plan: enough (tile, split) items to occupy every SM about twice, each split at least 2
// k-blocks deep, never more splits than k-blocks.
static void tc_plan(int tiles, int kblocks, int* splits, int* kbps) {
  int s = (2 * sm_count()) / tiles;
  if (s < 1) s = 1;
  int max_s = kblocks / 2 > 0 ? kblocks / 2 : 1;
  if (s > max_s) s = max_s;
  if (s > 32) s = 32;
  int per = ceil_div(kblocks, s);
  *kbps = per;
  *splits = ceil_div(kblocks, per);
}

bool tc_linear_supported(int m, int n, int k, int dtype) {
  if (m < 1 || m > 64 || n < 1 || encode_fn() == nullptr) return false;
  if (dtype == DT_BF16) return k >= 8 && (k % 8) == 0;
  if (dtype == DT_FP8) return k >= 16 && (k % 16) == 0;     // byte rows must be 16-byte multiples for TMA
  return false;
}

size_t tc_workspace_bytes(int m, int ld, int tiles, int k) {
  int s, kbps;
  tc_plan(tiles, ceil_div(k, TC_BK), &s, &kbps);
  return (size_t)s * m * ld * sizeof(float);
}

template <int M_PAD, int KIND>
static cudaError_t tc_launch_t(const TcParams& p, int grid, cudaStream_t st) {
  static bool attr_set[MAX_DEVICES] = {};
  cudaError_t e = ensure_dynamic_smem(gemm_tc_kernel<M_PAD, KIND>, TcSmem<M_PAD, KIND>::TOTAL, attr_set);
  if (e != cudaSuccess) return e;
  return launch_pdl(gemm_tc_kernel<M_PAD, KIND>, dim3(grid), dim3(KIND != TC_KIND_BF16 ? TC_THREADS_FP8 : TC_THREADS),
                    (size_t)TcSmem<M_PAD, KIND>::TOTAL, st, p);
}

template <int FP8>
static cudaError_t tc_launch_f(const TcParams& p, cudaStream_t st) {
  const int items = p.tile_begin[p.n_mats] * p.splits;
  const int grid = items < 2 * sm_count() ? items : 2 * sm_count();
  switch (pad_m(p.m)) {
    case 16: return tc_launch_t<16, FP8>(p, grid, st);
    case 32: return tc_launch_t<32, FP8>(p, grid, st);
    case 48: return tc_launch_t<48, FP8>(p, grid, st);
    default: return tc_launch_t<64, FP8>(p, grid, st);
  }
}

// A group of up to three bf16 matrices that share x and K, outputs side by side in one row of width ld.
//   mode PARTIAL: part[split][m][ld] (split-K sums left to the caller's reduce kernel); *splits_out tells how many
//   mode DIRECT : y[m][ld] = x w^T * scale + bias (+ y)   (forces one split)
//   mode SWIGLU : act[m][inter] = silu(x wg^T * sg) * (x wu^T * su)  (w[0] = gate, w[1] = up; one split)

cudaError_t tc_group_launch(const TcGroup& g, const TcOut& o, cudaStream_t st) {
  TcParams p;
  memset(&p, 0, sizeof(p));
  const int mode = o.mode;
  const int mp = pad_m(g.m);
  const int xkind = g.fp8 ? TM_F16 : TM_BF16;     // fp8 weights are widened to f16 and meet f16 activations
  const bool a8 = g.fp8 && g.a8;                  // ... unless the kernel quantises the activations to e4m3 itself
  if (a8 && (mode == TC_MODE_DIRECT || mode == TC_MODE_LOGITS)) return cudaErrorInvalidValue;
  if (a8 && (!o.amax_in || o.n_amax_in < 1)) return cudaErrorInvalidValue;
  if (!make_tmap(&p.tm_x, g.x, g.m, g.k, mp, xkind)) return cudaErrorInvalidValue;
  p.has_lo = (!g.fp8 && g.x_lo) ? 1 : 0;
  if (p.has_lo && !make_tmap(&p.tm_xl, g.x_lo, g.m, g.k, mp, xkind)) return cudaErrorInvalidValue;
  int tiles = 0, col = 0;
  for (int i = 0; i < g.n_mats; ++i) {
    if (!make_tmap(&p.tm_w[i], g.w[i], g.n[i], g.k, 64, a8 ? TM_E4M3_128 : (g.fp8 ? TM_E4M3 : TM_BF16))) return cudaErrorInvalidValue;
    p.n_out[i] = g.n[i];
    p.tile_begin[i] = tiles;
    p.out_col[i] = col;
    p.scale[i] = g.scale[i];
    p.bias[i] = g.bias[i];
    tiles += ceil_div(g.n[i], TC_BM);
    col += g.n[i];
  }
  p.n_mats = g.n_mats;
  p.kblocks = ceil_div(g.k, a8 ? 2 * TC_BK : TC_BK);
  p.m = g.m;
  p.amax_in = o.amax_in; p.n_amax_in = o.n_amax_in; p.amax_out = o.amax_out;
  p.mode = mode;
  p.status = o.status;
  p.stamp = o.stamp;
  p.ssq_in = o.ssq_in; p.nt_in = o.nt_in; p.inv_h = o.hidden > 0 ? 1.f / (float)o.hidden : 0.f; p.eps = o.eps;
  if (mode == TC_MODE_SWIGLU) {
    tiles = ceil_div(g.n[0], 64);      // one combined list of 64-feature tiles (gate + up rows interleaved)
    p.n_mats = 1;
    p.tile_begin[0] = 0; p.tile_begin[1] = tiles;
    p.splits = 1; p.kb_per_split = p.kblocks;
    p.act = o.act; p.act_lo_off = o.act_lo_off; p.act_fmt = o.act_fmt; p.inter = g.n[0];
  } else {
    p.tile_begin[g.n_mats] = tiles;
    if (mode == TC_MODE_PARTIAL) tc_plan(tiles, p.kblocks, &p.splits, &p.kb_per_split);
    else { p.splits = 1; p.kb_per_split = p.kblocks; }
    p.part = o.part; p.ldp = o.ld; p.y = o.y; p.ldy = o.ld; p.accumulate = o.accumulate;
    p.stats = (float4*)o.stats; p.mask_id = o.mask_id; p.write_logits = o.write_logits;
    if (mode == TC_MODE_PARTIAL && (size_t)p.splits * g.m * o.ld * sizeof(float) > o.part_bytes) return cudaErrorInvalidValue;
    if (mode == TC_MODE_LOGITS && (g.n_mats != 1 || !o.stats)) return cudaErrorInvalidValue;
  }
  if (o.splits_out) *o.splits_out = p.splits;
  return a8 ? tc_launch_f<TC_KIND_A8>(p, st) : (g.fp8 ? tc_launch_f<TC_KIND_FP8>(p, st) : tc_launch_f<TC_KIND_BF16>(p, st));
}

}  // namespace fdk
