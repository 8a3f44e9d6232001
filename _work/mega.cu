// Persistent forward kernel of the bf16 path (sm_100a): one cooperative launch runs every layer of one
// denoise / commit / prefill pass (Fast-dVLM Sec. 3.4; Appendix B Alg. 1 draft and verify passes).
//
// One CTA per SM.  Roles inside a CTA:
//   warp 0   weight producer: walks the whole forward's list of weight tiles owned by this CTA and keeps a
//            ring of 16 KB shared-memory stages full by TMA.  Weights do not depend on activations, so this
//            warp runs ahead across operator boundaries: while the CTA waits for other SMs, the next
//            operator's weights are already arriving.
//   warp 6   activation producer: waits (bounded) for the global counter that says the operator's input rows
//            are complete, then streams the matching activation k-blocks by TMA into a small second ring.
//   warp 1   MMA issuer: tcgen05.mma, weights = A operand (128 rows), block rows = N, fp32 accumulators in
//            tensor memory (two buffers).
//   warp 7   L2 prefetcher: while the latency-bound phases of a layer run (QKV, attention, O) HBM would idle, so
//            this warp asks for the layer's down-projection and O weights, its K/V cache rows and, later, the next
//            layer's QKV weights to be brought into L2 (each CTA a 1/grid share); one CTA then streams them at
//            L2 latency instead of DRAM latency.
//   warps 2-5 epilogue group: tcgen05.ld, split-K bookkeeping and the fused operator epilogues; the same four
//            warps run the attention items and the split-KV merge between the QKV and O projections.
//
// Work split ("stream-K"): an operator with T weight tiles of KB k-blocks is a line of T*KB units cut into
// gridDim.x equal contiguous shares, so every SM streams the same number of bytes.  A share that does not
// cover a whole tile leaves an fp32 partial in a per-CTA slot and bumps the tile's arrival counter; the CTA
// that arrives last sums the partials in CTA order (deterministic) and runs the epilogue:
//   QKV   folded RMSNorm factor, bias, rotary, q -> buffer, k / v -> cache rows L .. L + m - 1
//   O, D  residual add, next norm's gain folded into the bf16 copy, per-tile sum of squares
//   GU    SwiGLU -> bf16 activations
//   LM    logits (optional) and per-warp softmax statistics with the mask token excluded
// Operators are chained by monotonic global counters (release: fence + atomic add; acquire: ld.acquire).
// Every wait has an iteration / clock bound; a wait that gives up records a code in the status word, the CTA
// drains its bulk copies, frees its tensor memory and returns.
//
// The role loops are written with small iterator structs rather than lambdas: closures that captured the
// kernel parameter by reference were compiled into reads past the end of the parameter block.
#include <cuda.h>
#include <stdlib.h>

#include <mutex>

#include "attn_core.cuh"
#include "handle.h"
#include "tc_ptx.cuh"

namespace fdk {

constexpr int MG_THREADS = 256;
constexpr int MG_W_BYTES = 16384;        // one weight stage: 128 rows x 64 k bf16
constexpr long long MG_TIMEOUT = 1ll << 29;  // clock cycles (~0.3 s) before a global wait gives up
constexpr int MG_SMEM_LIMIT = 232448;    // 227 KB

enum { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_D = 3, OP_LM = 4 };
enum { MG_ERR_WPROD = 1, MG_ERR_XPROD = 2, MG_ERR_MMA = 3, MG_ERR_EPI = 4 };
// per-layer counter slots
enum { C_QKV = 0, C_ATT = 1, C_AO = 2, C_H2 = 3, C_ACT = 4, C_HOUT = 5, C_TILES = 8 };

// (tensor maps read from global memory by the TMA unit sit on 128-byte boundaries)
struct alignas(128) MgLayer {
  CUtensorMap tm_q, tm_k, tm_v, tm_o, tm_d;  // box {64 k, 128 rows}
  CUtensorMap tm_g, tm_u;                     // box {64 k, 16 rows}: gate / up rows interleaved per 16
  const float *bq, *bk, *bv, *g_attn, *g_mlp;
  bf16 *kc, *vc;                              // cache planes [Hkv][max_seq][d]
  const bf16 *wq, *wk, *wv, *wo, *wd;         // raw weight pointers (L2 prefetch)
};

// Tensor maps live in global memory (they are too many for the parameter block) ...
struct alignas(128) MgModel {
  CUtensorMap tm_lm;
};
static_assert(sizeof(MgLayer) % 128 == 0 && sizeof(CUtensorMap) == 128, "tensor maps must stay 128-byte aligned");

// ... everything else the kernel reads travels by value in the parameter block (constant bank): a field kept in
// global memory would have to be re-read after every global store of an epilogue loop.
struct MgConst {
  const MgLayer* layers;
  int n_layers, H, I, NQ, NKV, hq, hkv, d, vocab, mask_id, max_seq, nt;
  int R;               // rows allocated in the activation buffers (max_block)
  float eps, inv_h;
  const float* g_final;
  float* h;            // [R][H] residual stream
  bf16 *xg, *q, *ao, *act;
  float* ssq;          // [R][nt]
  const float2* cs;    // [R][d/2]
  float* part;         // [grid * 2][64][128] split-K partial slots
  float* att_o;
  float2* att_ml;
  float* logits;
  float4* stats;
  int* sync;
  int* status;
  int* trace;          // optional host-mapped words, one per role of CTA 0: (operator index << 8) | step last reached
  long long* tline;    // optional host-mapped timeline of one traced CTA: [operator][16] globaltimer stamps
  int trace_cta;
  int tq_begin[4];     // first tile of q, k, v; [3] = T_qkv
  int T_o, T_g, T_l, KB_h, KB_q, KB_i;
  int layer_stride, off_to, off_tg, off_td, off_lm;
  int op_sk[5], op_ge[5], op_off[5];   // per operator kind: K-splits per tile, participating CTAs, first CTA
};

struct MgRun {
  const MgModel* M;
  MgConst c;
  int m, L, causal;
  int lm_rows;         // 0: no LM head; 1: last row only; m: every row
  int write_logits;
  int qh, att_groups, chunk_keys, n_chunks;
};

// ---- work partition ----------------------------------------------------------------------------------
// An operator with T weight tiles of KB k-blocks is cut into W = T * SK units (unit j of a tile = k-blocks
// [j KB / SK, (j + 1) KB / SK)); the units form a line cut into Ge equal contiguous shares, one per participating
// CTA.  SK = 1 gives whole tiles (direct epilogue), SK = KB is stream-K (every SM streams the same bytes), a small
// SK is a classic split-K.  The Ge logical CTAs are spread over the grid: logical p runs on CTA (p G / Ge + off) % G.
struct Part {
  int T, KB, SK, Ge, off, G;
  __host__ __device__ long long W() const { return (long long)T * SK; }
  __host__ __device__ long long start(int p) const { return ((long long)p * W()) / Ge; }
  __host__ __device__ int owner(long long w) const { return (int)(((w + 1) * Ge - 1) / W()); }
  __host__ __device__ int kb_of(int j) const { return (int)(((long long)j * KB) / SK); }
  __host__ __device__ int phys(int p) const { return (int)((((long long)p * G) / Ge + off) % G); }
  // logical index of physical CTA c, or -1
  __host__ __device__ int logical(int c) const {
    const int cr = (c - off % G + G) % G;
    const int p = (int)(((long long)cr * Ge + G - 1) / G);
    return (p < Ge && (int)(((long long)p * G) / Ge) == cr) ? p : -1;
  }
};

// The segments (tile, k-blocks [kb0, kb1)) of one CTA's share.
struct SegIter {
  Part P;
  long long w, we;
  __device__ __forceinline__ SegIter(const Part& P_, int c) : P(P_) {
    const int p = P.logical(c);
    if (p >= 0) { w = P.start(p); we = P.start(p + 1); }
    else { w = 0; we = 0; }
  }
  __device__ __forceinline__ bool next(int& tile, int& kb0, int& kb1) {
    if (w >= we) return false;
    tile = (int)(w / P.SK);
    const int j0 = (int)(w - (long long)tile * P.SK);
    const long long left = we - w;
    const int j1 = (left < (long long)(P.SK - j0)) ? j0 + (int)left : P.SK;
    kb0 = P.kb_of(j0);
    kb1 = P.kb_of(j1);
    w += j1 - j0;
    return true;
  }
};

// The operators of one forward in launch order: per layer QKV, O, GU, D; then the LM head (layer index n_layers).
struct OpIter {
  int l, kind, n_layers, lm;
  __device__ __forceinline__ OpIter(int n_layers_, int lm_rows) : l(0), kind(-1), n_layers(n_layers_), lm(lm_rows > 0) {}
  __device__ __forceinline__ bool next() {
    if (l >= n_layers) return false;          // the LM head was the last one
    if (++kind > OP_D) { kind = OP_QKV; ++l; }
    if (l < n_layers) return true;
    if (!lm) return false;
    kind = OP_LM;
    return true;
  }
};

// ---- global-memory synchronisation ------------------------------------------------------------------
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void red_release_add(int* p, int v) {
  asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *p >= target.  False when the wait gave up or the CTA / grid is aborting.
__device__ __forceinline__ bool wait_count(const int* p, int target, volatile int* abort_flag, const int* status) {
  if (target <= 0) return true;
  if (ld_acquire(p) >= target) return true;
  const long long t0 = clock64();
  for (int it = 1;; ++it) {
    __nanosleep(64);               // a polling thread must not starve the warps that share its scheduler
    if (ld_acquire(p) >= target) return true;
    if (*abort_flag) return false;
    if ((it & 127) == 0 && (ld_relaxed(status) != 0 || clock64() - t0 > MG_TIMEOUT)) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 2, 128;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// A tensor map kept in global memory (written there by a host copy) has to be acquired by the thread that
// hands it to the TMA unit, which reads it through its own proxy.
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* tm) {
  asm volatile("fence.proxy.tensormap::generic.acquire.sys [%0], 128;" ::"l"(tm) : "memory");
}
// Ask for [p, p + bytes) (16-byte granules) to be brought into L2; no data returns to the SM.
__device__ __forceinline__ void l2_prefetch(const void* p, size_t bytes) {
  const char* c = (const char*)p;
  while (bytes > 0) {
    const uint32_t n = bytes > 32768 ? 32768u : (uint32_t)bytes;
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(c), "r"(n) : "memory");
    c += n;
    bytes -= n;
  }
}
// This CTA's share (by rows) of a row-major [rows][row_bytes] matrix.
__device__ __forceinline__ void l2_prefetch_rows(const void* base, int rows, size_t row_bytes, int cta, int G) {
  const int r0 = (int)(((long long)cta * rows) / G), r1 = (int)(((long long)(cta + 1) * rows) / G);
  if (r1 > r0) l2_prefetch((const char*)base + (size_t)r0 * row_bytes, (size_t)(r1 - r0) * row_bytes);
}
// Best-effort wait of the prefetch warp until this CTA has seen operator `op` start; false ends the prefetching.
__device__ __forceinline__ bool prefetch_wait(volatile int* cur_op, int op, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (*cur_op < op + 1) {
    if (*abort_flag || clock64() - t0 > TC_TIMEOUT) return false;
    __nanosleep(200);
  }
  return true;
}
__device__ __forceinline__ void trace_mark(const int* trace, int cta, int role, int op, int step) {
  if (trace && cta == 0) ((volatile int*)trace)[role] = (op << 8) | step;
}
// timeline slots per operator: 0 epilogue reaches the operator, 1 its attention done (O only), 2 first accumulator
// ready, 3 epilogue leaves the operator, 4 activation flag seen, 5 activation loads issued, 6 first MMA issued,
// 7 weight loads issued
__device__ __forceinline__ void tl_mark(long long* tl, bool on, int op, int slot) {
  if (tl && on) {
    long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    ((volatile long long*)tl)[op * 16 + slot] = t;
  }
}

// Shared memory: [weight ring][region R][barriers].  Region R holds the attention tiles while the epilogue group
// runs attention, and the activation ring plus the epilogues' exchange buffer while GEMMs run: the two never overlap
// in time inside a CTA (attention starts only after every QKV tile of the grid is finished, and the next
// activation load waits for the counter that every CTA bumps after its attention work).
template <int M_PAD, int D>
struct MgSmem {
  static constexpr int X_BYTES = M_PAD * 128;
  static constexpr int NX = M_PAD <= 32 ? 12 : (M_PAD <= 48 ? 8 : 5);       // activation ring stages
  static constexpr int XCH_OFF = NX * X_BYTES;                               // exchange buffer inside region R
  static constexpr int XCH_BYTES = ((M_PAD * 132 * 4 + 1023) / 1024) * 1024;
  static constexpr int GEMM_BYTES = XCH_OFF + XCH_BYTES;
  static constexpr int ATT_BYTES = attn_smem_bytes<D>() > GEMM_BYTES ? attn_smem_bytes<D>() : GEMM_BYTES;
  static constexpr int BAR_BYTES = 2048;
  static constexpr int NW_RAW = (MG_SMEM_LIMIT - 1024 - BAR_BYTES - ATT_BYTES) / MG_W_BYTES;
  static constexpr int NW = NW_RAW > 12 ? 12 : NW_RAW;
  static constexpr int W_OFF = 0;
  static constexpr int ATT_OFF = NW * MG_W_BYTES;
  static constexpr int X_OFF = ATT_OFF;
  static constexpr int BAR_OFF = ATT_OFF + ATT_BYTES;
  static constexpr int TOTAL = BAR_OFF + BAR_BYTES + 1024;
};

__device__ __forceinline__ Part op_part(const MgConst& M, int kind, int G) {
  Part g;
  switch (kind) {
    case OP_QKV: g.T = M.tq_begin[3]; g.KB = M.KB_h; break;
    case OP_O: g.T = M.T_o; g.KB = M.KB_q; break;
    case OP_GU: g.T = M.T_g; g.KB = M.KB_h; break;
    case OP_D: g.T = M.T_o; g.KB = M.KB_i; break;
    default: g.T = M.T_l; g.KB = M.KB_h; break;
  }
  g.SK = M.op_sk[kind]; g.Ge = M.op_ge[kind]; g.off = M.op_off[kind]; g.G = G;
  return g;
}

// ---- helpers of the epilogue group (128 threads, etid = index inside the group) ----------------------------
// group-wide bounded wait on a global counter: one thread polls, the result is broadcast
__device__ __forceinline__ bool group_wait(const int* flag, int target, int etid, volatile int* s_flag, volatile int* abort_flag,
                                           const int* status) {
  if (etid == 0) *s_flag = wait_count(flag, target, abort_flag, status) ? 1 : 0;
  epi_bar();
  const bool r = *s_flag != 0;
  epi_bar();
  return r;
}
// release: every thread's stores are ordered before the barrier; one thread then fences (cumulative) and bumps the
// counter.  Each thread orders its own generic stores ahead of later async-proxy (TMA) reads of the same rows.
__device__ __forceinline__ void group_signal(int* flag, int etid) {
  fence_proxy_async_all();
  epi_bar();
  if (etid == 0) {
    __threadfence();
    red_release_add(flag, 1);
  }
}
// s_rstd[i] = rsqrt(mean(h[row0 + i]^2) + eps) from the per-tile sums of squares
__device__ __forceinline__ void load_rstd(const float* ssq, int nt, float inv_h, float eps, float* s_rstd, int row0, int rows,
                                          int etid) {
  if (etid < rows) {
    const float* p = ssq + (size_t)(row0 + etid) * nt;
    float s = 0.f;
    for (int t0 = 0; t0 < nt; t0 += 8) {         // eight independent loads in flight, summed in index order
      float r[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) r[i] = (t0 + i < nt) ? __ldcg(p + t0 + i) : 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) s += r[i];
    }
    s_rstd[etid] = rsqrtf(s * inv_h + eps);
  }
  epi_bar();
}

template <int M_PAD, int D>
__global__ void __launch_bounds__(MG_THREADS, 1) forward_mega_kernel(const MgRun Rp) {
  using S = MgSmem<M_PAD, D>;
  constexpr int NW = S::NW, MG_NX = S::NX;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t bar0 = base + S::BAR_OFF;
  // barrier slots (8 bytes each)
  const uint32_t w_full0 = bar0, w_empty0 = bar0 + 8u * NW, x_full0 = bar0 + 8u * (2 * NW), x_empty0 = bar0 + 8u * (2 * NW + MG_NX);
  const uint32_t t_full0 = bar0 + 8u * (2 * NW + 2 * MG_NX), t_empty0 = t_full0 + 16u;
  constexpr int MISC = 8 * (2 * 12 + 2 * 12 + 4);   // past the largest barrier set
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(sm + S::BAR_OFF + MISC);
  volatile int* abort_flag = (volatile int*)(sm + S::BAR_OFF + MISC + 8);
  volatile int* s_flag = (volatile int*)(sm + S::BAR_OFF + MISC + 16);     // epilogue group broadcast word
  volatile int* s_cur_op = (volatile int*)(sm + S::BAR_OFF + MISC + 24);   // 1 + index of the operator whose inputs are ready
  float* s_rstd = (float*)(sm + S::BAR_OFF + MISC + 32);                    // [64]
  float* s_red = s_rstd + 64;                                               // [4][M_PAD <= 64]
  float* s_xch = (float*)(sm + S::ATT_OFF + S::XCH_OFF);                                 // [M_PAD][<=132] exchange (GEMM epilogues only)

  // the run description in registers
  const MgModel* const Mp = Rp.M;
  const int r_m = Rp.m, r_L = Rp.L, r_causal = Rp.causal, r_lm_rows = Rp.lm_rows, r_write_logits = Rp.write_logits;
  const int r_qh = Rp.qh, r_groups = Rp.att_groups, r_chunk_keys = Rp.chunk_keys, r_n_chunks = Rp.n_chunks;
  const MgModel& M = *Mp;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, G = gridDim.x;
  // Two accumulator buffers of NACC accumulators each: the NACC K sub-steps of a k-block go to different accumulators,
  // so consecutive MMAs do not wait for one another's accumulate (with N <= 64 an MMA is far shorter than its latency).
  constexpr int NACC = TC_BK / 16;
  constexpr int ACC_COLS = NACC * M_PAD;
  constexpr int TMEM_COLS = (2 * ACC_COLS <= 128) ? 128 : ((2 * ACC_COLS <= 256) ? 256 : 512);

  if (threadIdx.x == 0) {
    for (int s = 0; s < NW; ++s) { mbar_init(w_full0 + 8u * s, 1); mbar_init(w_empty0 + 8u * s, 1); }
    for (int s = 0; s < MG_NX; ++s) { mbar_init(x_full0 + 8u * s, 1); mbar_init(x_empty0 + 8u * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(t_full0 + 8u * a, 1); mbar_init(t_empty0 + 8u * a, 4); }
    *abort_flag = 0;
    *s_cur_op = 0;
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
  int* const sync = Rp.c.sync;
  const int* const status = Rp.c.status;
  const int* const trace = Rp.c.trace;
  long long* const tl = Rp.c.tline;
  const bool tl_on = (cta == Rp.c.trace_cta);
  const int n_layers = Rp.c.n_layers, layer_stride = Rp.c.layer_stride, T_o = Rp.c.T_o, T_g = Rp.c.T_g;

  if (warp == 0) {
    // =========================================== weight producer ===========================================
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first();
      int stage = 0;
      uint32_t phase = 0, armed = 0, armed_parity = 0;
      bool ok = true;
      OpIter ops(n_layers, r_lm_rows);
      while (ok && ops.next()) {
        const int kind = ops.kind, l = ops.l;
        const Part g = op_part(Rp.c, kind, G);
        const MgLayer* Ly = &Rp.c.layers[kind == OP_LM ? 0 : l];
        trace_mark(trace, cta, 0, l * 4 + kind, 1);
        switch (kind) {
          case OP_QKV: tensormap_acquire(&Ly->tm_q); tensormap_acquire(&Ly->tm_k); tensormap_acquire(&Ly->tm_v); break;
          case OP_O: tensormap_acquire(&Ly->tm_o); break;
          case OP_GU: tensormap_acquire(&Ly->tm_g); tensormap_acquire(&Ly->tm_u); break;
          case OP_D: tensormap_acquire(&Ly->tm_d); break;
          default: tensormap_acquire(&M.tm_lm); break;
        }
        SegIter seg(g, cta);
        int tile, kb0, kb1;
        while (ok && seg.next(tile, kb0, kb1)) {
          const CUtensorMap* tm = &M.tm_lm;
          int r0 = tile * TC_BM;
          if (kind == OP_QKV) {
            int mi = 0;
            while (mi < 2 && tile >= Rp.c.tq_begin[mi + 1]) ++mi;
            tm = mi == 0 ? &Ly->tm_q : (mi == 1 ? &Ly->tm_k : &Ly->tm_v);
            r0 = (tile - Rp.c.tq_begin[mi]) * TC_BM;
          } else if (kind == OP_O) tm = &Ly->tm_o;
          else if (kind == OP_D) tm = &Ly->tm_d;
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(w_empty0 + 8u * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
            const uint32_t dst = base + S::W_OFF + stage * MG_W_BYTES;
            const uint32_t fb = w_full0 + 8u * stage;
            mbar_expect_tx(fb, MG_W_BYTES);
            armed |= 1u << stage;
            armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
            if (kind == OP_GU) {
              // 64 features per tile: lane quarter qq of the accumulator holds gate rows of features 16qq .. 16qq+15
              // in its lanes 0..15 and the matching up rows in lanes 16..31
#pragma unroll
              for (int qq = 0; qq < 4; ++qq) {
                tma_load_2d(dst + (32 * qq) * 128, &Ly->tm_g, fb, kb * TC_BK, tile * 64 + 16 * qq, pol_w);
                tma_load_2d(dst + (32 * qq + 16) * 128, &Ly->tm_u, fb, kb * TC_BK, tile * 64 + 16 * qq, pol_w);
              }
            } else {
              tma_load_2d(dst, tm, fb, kb * TC_BK, r0, pol_w);
            }
            if (++stage == NW) { stage = 0; phase ^= 1u; }
          }
        }
        tl_mark(tl, tl_on, l * 4 + kind, 7);
      }
      if (!ok) {
        atomicCAS(Rp.c.status, 0, MG_ERR_WPROD);
        for (int s = 0; s < NW; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t par = (armed_parity >> s) & 1u;
          const long long t0 = clock64();
          while (!mbar_try_wait(w_full0 + 8u * s, par) && clock64() - t0 < TC_TIMEOUT) {}
        }
      }
    }
  } else if (warp == 6) {
    // ========================================= activation producer =========================================
    // The whole warp copies the [M_PAD x 64] bf16 activation tile of each k-block from L2 with plain 16-byte loads
    // and writes it in the 128-byte-swizzled layout the MMA expects.  (Bulk tensor copies of these small,
    // latency-critical tiles would queue behind the weight stream in the SM's copy engine.)
    bool ok = true;
    int stage = 0;
    uint32_t phase = 0;
    constexpr int CPL = M_PAD * 8 / 32;        // 16-byte chunks per lane and tile
    OpIter ops(n_layers, r_lm_rows);
    while (ok && ops.next()) {
      const int kind = ops.kind, l = ops.l;
      const Part g = op_part(Rp.c, kind, G);
      const int* lc = sync + (size_t)(kind == OP_LM ? l - 1 : l) * layer_stride;
      const bf16* xb = Rp.c.xg;
      int K = Rp.c.H;
      const int* flag = lc;
      int target = 0, row0 = 0;
      switch (kind) {
        case OP_QKV: if (l > 0) { flag = lc - layer_stride + C_HOUT; target = T_o; } break;
        case OP_O: xb = Rp.c.ao; K = Rp.c.NQ; flag = lc + C_AO; target = G; break;
        case OP_GU: flag = lc + C_H2; target = T_o; break;
        case OP_D: xb = Rp.c.act; K = Rp.c.I; flag = lc + C_ACT; target = T_g; break;
        default: flag = lc + C_HOUT; target = T_o; row0 = r_m - r_lm_rows; break;
      }
      if (lane == 0) {
        trace_mark(trace, cta, 1, l * 4 + kind, 1);
        ok = wait_count(flag, target, abort_flag, status);
        trace_mark(trace, cta, 1, l * 4 + kind, 2);
        tl_mark(tl, tl_on, l * 4 + kind, 4);
        *s_cur_op = l * 4 + kind + 1;
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      __syncwarp();                                        // lane 0's acquire orders the whole warp's loads below
      if (!ok) break;
      // k-blocks are handled NB at a time: all their loads are in flight together (one L2 round trip per group),
      // and only the stores wait for free stages
      constexpr int NB = (32 / CPL) < 2 ? 2 : (32 / CPL);
      SegIter seg(g, cta);
      int tile, kb0 = 0, kb1 = 0;
      bool more = true;
      int ngrp = 0;
      if (lane == 0) tl_mark(tl, tl_on, l * 4 + kind, 12);
      while (ok && more) {
        int kbs[NB];
        int n = 0;
        while (n < NB) {
          if (kb0 >= kb1 && !seg.next(tile, kb0, kb1)) { more = false; break; }
          kbs[n++] = kb0++;
        }
        if (n == 0) break;
        uint4 val[NB][CPL];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
#pragma unroll
          for (int i = 0; i < CPL; ++i) {
            const int ch = lane + 32 * i, r = ch >> 3, c = ch & 7;
            const int col = kbs[j < n ? j : 0] * TC_BK + c * 8;
            const bool valid = j < n && (row0 + r) < Rp.c.R && col < K;
            val[j][i] = valid ? __ldcg(reinterpret_cast<const uint4*>(xb + (size_t)(row0 + r) * K + col)) : make_uint4(0u, 0u, 0u, 0u);
          }
        }
        if (lane == 0 && ngrp == 0) { tl_mark(tl, tl_on && (val[0][0].x != 0x12345u), l * 4 + kind, 13); }
#pragma unroll
        for (int j = 0; j < NB; ++j) {
          if (j < n) {                                      // uniform across the warp
            if (lane == 0) ok = mbar_wait(x_empty0 + 8u * stage, phase ^ 1u, abort_flag);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (ok) {
              const uint32_t dst = base + S::X_OFF + stage * S::X_BYTES;
#pragma unroll
              for (int i = 0; i < CPL; ++i) {
                const int ch = lane + 32 * i, r = ch >> 3, c = ch & 7;
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + r * 128 + ((c ^ (r & 7)) << 4)), "r"(val[j][i].x),
                             "r"(val[j][i].y), "r"(val[j][i].z), "r"(val[j][i].w) : "memory");
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> the MMA's async-proxy reads
              __syncwarp();
              if (lane == 0) mbar_arrive(x_full0 + 8u * stage);
              if (++stage == MG_NX) { stage = 0; phase ^= 1u; }
            }
          }
        }
        if (lane == 0 && ngrp == 0) tl_mark(tl, tl_on, l * 4 + kind, 14);
        ++ngrp;
      }
      if (lane == 0) tl_mark(tl, tl_on, l * 4 + kind, 5);
    }
    if (!ok && lane == 0) atomicCAS(Rp.c.status, 0, MG_ERR_XPROD);
  } else if (warp == 7) {
    // ============================================== L2 prefetcher ============================================
    if (lane == 0) {
      const size_t rb_h = (size_t)Rp.c.H * 2, rb_q = (size_t)Rp.c.NQ * 2, rb_i = (size_t)Rp.c.I * 2;
      for (int l = 0; l < n_layers; ++l) {
        const MgLayer* Ly = &Rp.c.layers[l];
        if (!prefetch_wait(s_cur_op, l * 4 + OP_QKV, abort_flag)) break;
        l2_prefetch_rows(Ly->wo, Rp.c.H, rb_q, cta, G);
        for (int hk = 0; hk < Rp.c.hkv; ++hk) {
          l2_prefetch_rows(Ly->kc + (size_t)hk * Rp.c.max_seq * D, r_L, (size_t)D * 2, cta, G);
          l2_prefetch_rows(Ly->vc + (size_t)hk * Rp.c.max_seq * D, r_L, (size_t)D * 2, cta, G);
        }
        l2_prefetch_rows(Ly->wd, Rp.c.H, rb_i, cta, G);
        if (l + 1 < n_layers) {
          if (!prefetch_wait(s_cur_op, l * 4 + OP_GU, abort_flag)) break;
          const MgLayer* Ln = &Rp.c.layers[l + 1];
          l2_prefetch_rows(Ln->wq, Rp.c.NQ, rb_h, cta, G);
          l2_prefetch_rows(Ln->wk, Rp.c.NKV, rb_h, cta, G);
          l2_prefetch_rows(Ln->wv, Rp.c.NKV, rb_h, cta, G);
        }
      }
    }
  } else if (warp == 1) {
    // ============================================== MMA issuer ==============================================
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(M_PAD);
      int ws = 0, xs = 0, nseg = 0;
      uint32_t wph = 0, xph = 0;
      bool ok = true;
      OpIter ops(n_layers, r_lm_rows);
      while (ok && ops.next()) {
        const int kind = ops.kind, l = ops.l;
        trace_mark(trace, cta, 2, l * 4 + kind, 1);
        const Part g = op_part(Rp.c, kind, G);
        SegIter seg(g, cta);
        int tile, kb0, kb1;
        while (ok && seg.next(tile, kb0, kb1)) {
          const int acc = nseg & 1;
          const uint32_t acc_phase = (uint32_t)(nseg >> 1) & 1u;
          ++nseg;
          if (!mbar_wait(t_empty0 + 8u * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * ACC_COLS);
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(w_full0 + 8u * ws, wph, abort_flag) || !mbar_wait(x_full0 + 8u * xs, xph, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (kb == kb0) tl_mark(tl, tl_on, l * 4 + kind, 6);
            const uint64_t adesc = umma_desc_sw128(base + S::W_OFF + ws * MG_W_BYTES);
            const uint64_t bdesc = umma_desc_sw128(base + S::X_OFF + xs * S::X_BYTES);
#pragma unroll
            for (int kk = 0; kk < TC_BK / 16; ++kk)
              umma_bf16(d_tmem + (uint32_t)(kk * M_PAD), adesc + 2u * kk, bdesc + 2u * kk, idesc, (kb > kb0) ? 1u : 0u);
            umma_commit(w_empty0 + 8u * ws);
            umma_commit(x_empty0 + 8u * xs);
            if (++ws == NW) { ws = 0; wph ^= 1u; }
            if (++xs == MG_NX) { xs = 0; xph ^= 1u; }
          }
          if (ok) umma_commit(t_full0 + 8u * acc);
        }
      }
      if (!ok) atomicCAS(Rp.c.status, 0, MG_ERR_MMA);
    }
  } else {
    // ================================ epilogue group (warps 2..5, 128 threads) ================================
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const int et = q * 32 + lane;                 // accumulator row held by this thread (0..127)
    const int etid = (warp - 2) * 32 + lane;      // index inside the group
    const int nt = Rp.c.nt, hq = Rp.c.hq, hkv = Rp.c.hkv, max_seq = Rp.c.max_seq, H = Rp.c.H, I = Rp.c.I, vocab = Rp.c.vocab, mask_id = Rp.c.mask_id;
    const float inv_h = Rp.c.inv_h, eps = Rp.c.eps;
    int nseg = 0;
    bool ok = true;
    OpIter ops(n_layers, r_lm_rows);
    while (ok && ops.next()) {
      const int kind = ops.kind, l = ops.l;
      const Part g = op_part(Rp.c, kind, G);
      int* lc = sync + (size_t)(kind == OP_LM ? l - 1 : l) * layer_stride;
      const MgLayer* Ly = &Rp.c.layers[kind == OP_LM ? 0 : l];
      // per-layer pointers of this operator, read once (the layer table is in global memory)
      bf16* const kc = Ly->kc;
      bf16* const vc = Ly->vc;
      const float* const bq = (kind == OP_QKV) ? Ly->bq : nullptr;
      const float* const bk = (kind == OP_QKV) ? Ly->bk : nullptr;
      const float* const bv = (kind == OP_QKV) ? Ly->bv : nullptr;
      const float* const res_gain = (kind == OP_O) ? Ly->g_mlp
                                    : (kind == OP_D ? (l + 1 < n_layers ? Rp.c.layers[l + 1].g_attn : Rp.c.g_final) : nullptr);
      const int m = (kind == OP_LM) ? r_lm_rows : r_m;
      const int xrow0 = (kind == OP_LM) ? r_m - r_lm_rows : 0;
      if (etid == 0) { trace_mark(trace, cta, 3, l * 4 + kind, 1); tl_mark(tl, tl_on, l * 4 + kind, 0); }

      if (kind == OP_O) {
        // ---------------- attention of this layer: split-KV items, then the merge of the key chunks ----------------
        if (!group_wait(lc + C_QKV, Rp.c.tq_begin[3], etid, s_flag, abort_flag, status)) { ok = false; break; }
        const int n_items = hkv * r_groups * r_n_chunks;
        for (int item = cta; item < n_items; item += G) {
          const int chunk = item % r_n_chunks, rest = item / r_n_chunks;
          const int grp = rest % r_groups, hk = rest / r_groups;
          attn_item<D>(Rp.c.q, kc, vc, Rp.c.att_o, Rp.c.att_ml, r_m, r_L, max_seq, hq, hkv, r_qh, r_chunk_keys, r_n_chunks,
                       r_causal, chunk, grp, hk, base + S::ATT_OFF, etid);
        }
        if (etid == 0) trace_mark(trace, cta, 3, l * 4 + kind, 2);
        group_signal(lc + C_ATT, etid);
        if (!group_wait(lc + C_ATT, G, etid, s_flag, abort_flag, status)) { ok = false; break; }
        if (etid == 0) trace_mark(trace, cta, 3, l * 4 + kind, 3);
        // one warp per (row, head): the CTA's four warps take consecutive pairs
        for (int p = cta * 4 + (warp - 2); p < r_m * hq; p += G * 4) {
          const int i = p / hq, head = p % hq;
          attn_merge_warp<D>(Rp.c.att_o, Rp.c.att_ml, Rp.c.ao + ((size_t)i * hq + head) * D, ((size_t)head * r_m + i) * r_n_chunks, r_n_chunks, lane);
        }
        group_signal(lc + C_AO, etid);
        if (etid == 0) { trace_mark(trace, cta, 3, l * 4 + kind, 4); tl_mark(tl, tl_on, l * 4 + kind, 1); }
      }

      // the folded RMSNorm factor of this operator's input rows (QKV, GU, LM) is loaded before the first epilogue
      bool have_rstd = false;
      (void)have_rstd;
      const int* rstd_flag = (kind == OP_QKV) ? lc - layer_stride + C_HOUT : (kind == OP_GU ? lc + C_H2 : lc + C_HOUT);
      const int rstd_target = (kind == OP_QKV && l == 0) ? 0 : T_o;
      const bool wants_rstd = (kind == OP_QKV || kind == OP_GU || kind == OP_LM);

      SegIter seg(g, cta);
      int tile, kb0, kb1;
      const bool is_resid = (kind == OP_O || kind == OP_D);
      if (seg.w < seg.we) {
        // inputs of the epilogues that do not depend on this operator's own MMAs are fetched while those run
        if (wants_rstd) {
          if (!group_wait(rstd_flag, rstd_target, etid, s_flag, abort_flag, status)) { ok = false; break; }
          load_rstd(Rp.c.ssq, nt, inv_h, eps, s_rstd, xrow0, m, etid);
          have_rstd = true;
        } else if (is_resid) {
          // the residual rows this operator adds to: complete once the previous residual operator has finished
          const int* hflag = (kind == OP_O) ? lc - layer_stride + C_HOUT : lc + C_H2;
          if (!group_wait(hflag, (kind == OP_O && l == 0) ? 0 : T_o, etid, s_flag, abort_flag, status)) { ok = false; break; }
        }
      }
      while (ok && seg.next(tile, kb0, kb1)) {
        const int acc = nseg & 1;
        const uint32_t acc_phase = (uint32_t)(nseg >> 1) & 1u;
        ++nseg;
        // epilogue inputs that do not depend on the MMAs: residual rows (O, D) or the rotary table entries (QKV)
        constexpr bool PRE_CS = (M_PAD <= 32);
        float pre[PRE_CS ? 2 * M_PAD : M_PAD];
        float pre_gain = 0.f;
        if (is_resid) {
          const int c = tile * TC_BM + et;
          pre_gain = (c < H) ? res_gain[c] : 0.f;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) pre[b] = (c < H && b < m) ? __ldcg(&Rp.c.h[(size_t)b * H + c]) : 0.f;
        } else if (PRE_CS && kind == OP_QKV) {
          const int jq = et % (D / 2);
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) {
            const float2 c2 = Rp.c.cs[(b < m ? b : 0) * (D / 2) + jq];
            pre[(2 * b) % (PRE_CS ? 2 * M_PAD : M_PAD)] = c2.x;
            pre[(2 * b + 1) % (PRE_CS ? 2 * M_PAD : M_PAD)] = c2.y;
          }
        }
        if (etid == 0) *s_flag = mbar_wait(t_full0 + 8u * acc, acc_phase, abort_flag) ? 1 : 0;
        epi_bar();
        if (*s_flag == 0) { ok = false; break; }
        if (etid == 0) { trace_mark(trace, cta, 3, l * 4 + kind, 5); tl_mark(tl, tl_on, l * 4 + kind, 2); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float v[M_PAD];
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * ACC_COLS);
#pragma unroll
        for (int c = 0; c < M_PAD; c += 16) tmem_ld16(taddr + c, v + c);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int a = 1; a < NACC; ++a) {                 // sum of the K sub-step accumulators, fixed order
          float t[M_PAD];
#pragma unroll
          for (int c = 0; c < M_PAD; c += 16) tmem_ld16(taddr + (uint32_t)(a * M_PAD + c), t + c);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int i = 0; i < M_PAD; ++i) v[i] += t[i];
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(t_empty0 + 8u * acc);
        if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 8);

        // ---- split tile: leave a partial; the last CTA to arrive sums all partials in CTA order ----
        if (!(kb0 == 0 && kb1 == g.KB)) {
          const int me = g.logical(cta);
          const int first_tile = (int)(g.start(me) / g.SK);
          float* mine = Rp.c.part + ((size_t)(cta * 2 + (tile == first_tile ? 0 : 1)) * 64) * 128;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b)
            if (b < m) mine[b * 128 + et] = v[b];
          epi_bar();
          const int cf = g.owner((long long)tile * g.SK), cl = g.owner((long long)tile * g.SK + g.SK - 1);
          int* tcnt = lc + (kind == OP_LM ? Rp.c.off_lm : (kind == OP_QKV ? (int)C_TILES : (kind == OP_O ? Rp.c.off_to : (kind == OP_GU ? Rp.c.off_tg : Rp.c.off_td)))) + tile;
          // one acq_rel atomic after the barrier: releases every thread's partial stores (cumulative) and, for the
          // last arriver, acquires the other CTAs' partials for the whole group (through the second barrier)
          if (etid == 0) *s_flag = (atom_add_acq_rel(tcnt, 1) == cl - cf) ? 1 : 0;
          epi_bar();
          const bool last = *s_flag != 0;
          epi_bar();                               // s_flag may be rewritten from here on
          if (!last) continue;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) v[b] = 0.f;
          constexpr int CU = (M_PAD <= 16) ? 4 : (M_PAD <= 32 ? 2 : 1);   // partials loaded together (register budget)
          for (int c2 = cf; c2 <= cl; c2 += CU) {
            float pv[CU][M_PAD];
#pragma unroll
            for (int u2 = 0; u2 < CU; ++u2) {
              const int c3 = (c2 + u2 <= cl) ? c2 + u2 : cl;
              const int ft = (int)(g.start(c3) / g.SK);
              const float* src = Rp.c.part + ((size_t)(g.phys(c3) * 2 + (tile == ft ? 0 : 1)) * 64) * 128;
#pragma unroll
              for (int b = 0; b < M_PAD; ++b) pv[u2][b] = (b < m) ? __ldcg(&src[b * 128 + et]) : 0.f;
            }
#pragma unroll
            for (int u2 = 0; u2 < CU; ++u2) {
              if (c2 + u2 <= cl) {                 // summed in CTA order
#pragma unroll
                for (int b = 0; b < M_PAD; ++b) v[b] += pv[u2][b];
              }
            }
          }
        }

        if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 9);
        // ---- operator epilogue on a complete tile: v[b] = sum_k w[row et of the tile][k] x[b][k] ----
        if (kind == OP_QKV) {
          int mi = 0;
          while (mi < 2 && tile >= Rp.c.tq_begin[mi + 1]) ++mi;
          const int n = (tile - Rp.c.tq_begin[mi]) * TC_BM + et;          // feature inside its matrix
          const int n_out = (mi == 0) ? Rp.c.NQ : Rp.c.NKV;
          const bool in_range = n < n_out;
          const float* bias = (mi == 0) ? bq : (mi == 1 ? bk : bv);
          const float bi = (in_range && bias) ? bias[n] : 0.f;
          const int head = n / D, j = n % D;
          constexpr int half = D / 2;
          const bool lo = j < half;
          const int jj = lo ? j : j - half;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) v[b] = v[b] * s_rstd[b < m ? b : 0] + bi;
          if (mi < 2) {
            // rotary: the partner feature j +- d/2 sits in another warp's rows -> exchange through shared memory
#pragma unroll
            for (int b = 0; b < M_PAD; ++b) s_xch[b * 128 + et] = v[b];
            epi_bar();
            const int pt = lo ? et + half : et - half;
#pragma unroll
            for (int b = 0; b < M_PAD; ++b) {
              if (b < m) {
                const float other = s_xch[b * 128 + pt];
                float2 c;
                if (PRE_CS) { c.x = pre[(2 * b) % (PRE_CS ? 2 * M_PAD : M_PAD)]; c.y = pre[(2 * b + 1) % (PRE_CS ? 2 * M_PAD : M_PAD)]; }
                else c = Rp.c.cs[b * half + jj];
                v[b] = lo ? v[b] * c.x - other * c.y : v[b] * c.x + other * c.y;
              }
            }
            epi_bar();
          }
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 10);
          if (in_range) {
            bf16* dst;
            size_t stride;
            if (mi == 0) { dst = Rp.c.q + (size_t)head * D + j; stride = (size_t)hq * D; }
            else { dst = (mi == 1 ? kc : vc) + ((size_t)head * max_seq + r_L) * D + j; stride = D; }
#pragma unroll
            for (int b = 0; b < M_PAD; ++b)
              if (b < m) dst[(size_t)b * stride] = __float2bfloat16_rn(v[b]);
          }
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 1);
          group_signal(lc + C_QKV, etid);
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 11);
        } else if (kind == OP_O || kind == OP_D) {
          const int c = tile * TC_BM + et;
          const bool in_range = c < H;
          const float gn = pre_gain;
          // squares go through shared memory ([row][132]: 4 x 33 per row, conflict-free both ways) for the per-row sums
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) {
            if (b < m) {                                   // uniform across the group
              const float hv = pre[b] + v[b];
              if (in_range) {
                const size_t idx = (size_t)b * H + c;
                Rp.c.h[idx] = hv;
                Rp.c.xg[idx] = __float2bfloat16_rn(hv * gn);
              }
              s_xch[b * 132 + (warp - 2) * 33 + lane] = in_range ? hv * hv : 0.f;
            }
          }
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 10);
          epi_bar();
          for (int w4 = etid; w4 < m * 4; w4 += 128) {
            const int b = w4 >> 2, part = w4 & 3;
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) ss += s_xch[b * 132 + part * 33 + i];
            s_red[part * M_PAD + b] = ss;
          }
          epi_bar();
          if (etid < m) Rp.c.ssq[(size_t)etid * nt + tile] = s_red[etid] + s_red[M_PAD + etid] + s_red[2 * M_PAD + etid] + s_red[3 * M_PAD + etid];
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 1);
          group_signal(lc + (kind == OP_O ? C_H2 : C_HOUT), etid);
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 11);
        } else if (kind == OP_GU) {
          const int col = tile * 64 + q * 16 + (lane & 15);
          const bool live = lane < 16 && col < I;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) {
            const float other = __shfl_xor_sync(0xffffffffu, v[b], 16);   // lanes 0..15: the matching "up" value
            if (live && b < m) {
              const float rs = s_rstd[b];
              const float gt = v[b] * rs;
              Rp.c.act[(size_t)b * I + col] = __float2bfloat16_rn(gt / (1.f + __expf(-gt)) * (other * rs));
            }
          }
          if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 1);
          group_signal(lc + C_ACT, etid);
        } else {
          const int n = tile * TC_BM + et;                    // vocabulary id held by this thread
          const bool in_range = n < vocab;
          const bool counted = in_range && n != mask_id;
#pragma unroll
          for (int b = 0; b < M_PAD; ++b) {
            if (b >= m) break;                                // uniform across the group
            const float lg = v[b] * s_rstd[b];
            if (r_write_logits && in_range) Rp.c.logits[(size_t)b * vocab + n] = lg;
            float mx = counted ? lg : -INFINITY;
            int ix = counted ? n : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const float omx = __shfl_xor_sync(0xffffffffu, mx, o);
              const int oix = __shfl_xor_sync(0xffffffffu, ix, o);
              if (omx > mx || (omx == mx && oix < ix)) { mx = omx; ix = oix; }
            }
            float e = (counted && mx > -INFINITY) ? __expf(lg - mx) : 0.f;
            e = warp_sum(e);
            if (lane == 0) Rp.c.stats[(size_t)(tile * 4 + q) * m + b] = make_float4(mx, e, __int_as_float(ix), 0.f);
          }
        }
      }
      if (etid == 0) tl_mark(tl, tl_on, l * 4 + kind, 3);
    }
    if (!ok && etid == 0) atomicCAS(Rp.c.status, 0, MG_ERR_EPI);
  }

  // ---- teardown: every thread arrives here, whatever happened ----
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ================================================================================================
// host side
// ================================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn mg_encode_fn() {
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
// 2-D bf16 row-major [rows, cols], box {64 columns, box_rows}, 128-byte swizzle, zero fill outside.
static bool mg_tmap(CUtensorMap* tm, const void* ptr, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = mg_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct MegaCtx {
  MgModel* d_model = nullptr;
  MgLayer* d_layers = nullptr;
  int* d_sync = nullptr;
  float* d_part = nullptr;
  float* d_att_o = nullptr;
  float2* d_att_ml = nullptr;
  size_t sync_bytes = 0;
  MgConst cst;              // by-value part of the kernel parameter
  int* h_trace = nullptr;   // host-mapped, only with FDVLM_MEGA_TRACE=1
  long long* h_tline = nullptr;
  int n_ops = 0;
  int grid = 0;
};

struct MgAttPlan { int qh, groups, chunk_keys, n_chunks; };
static MgAttPlan mg_att_plan(int n, int T, int hq, int hkv, int G) {
  const int Gh = hq / hkv;
  MgAttPlan p;
  p.qh = 1;
  for (int c = Gh; c >= 1; --c)
    if (c * n <= AT_ROWS) { p.qh = c; break; }
  p.groups = ceil_div(Gh, p.qh);
  const int per_chunk = hkv * p.groups;
  const int tiles = ceil_div(T, AT_KEYS);
  int want = G / per_chunk;
  if (want > tiles) want = tiles;
  if (want < 1) want = 1;
  p.chunk_keys = ceil_div(tiles, want) * AT_KEYS;
  p.n_chunks = ceil_div(T, p.chunk_keys);
  return p;
}

template <int M_PAD, int D>
static cudaError_t mg_launch_t(const MgRun& run, int grid, cudaStream_t st) {
  using S = MgSmem<M_PAD, D>;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(forward_mega_kernel<M_PAD, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  void* args[] = {(void*)&run};
  return cudaLaunchCooperativeKernel((const void*)forward_mega_kernel<M_PAD, D>, dim3(grid), dim3(MG_THREADS), args, S::TOTAL, st);
}

template <int D>
static cudaError_t mg_launch_d(const MgRun& run, int grid, cudaStream_t st) {
  const int mp = run.m <= 16 ? 16 : (run.m <= 32 ? 32 : (run.m <= 48 ? 48 : 64));
  switch (mp) {
    case 16: return mg_launch_t<16, D>(run, grid, st);
    case 32: return mg_launch_t<32, D>(run, grid, st);
    case 48: return mg_launch_t<48, D>(run, grid, st);
    default: return mg_launch_t<64, D>(run, grid, st);
  }
}

void mega_destroy(fdvlm_t* h) {
  MegaCtx* c = (MegaCtx*)h->mega;
  if (!c) return;
  if (c->h_trace) {
    fprintf(stderr, "fdvlm persistent kernel trace (CTA 0; op<<8|step): wprod %x  xprod %x  mma %x  epi %x\n", c->h_trace[0],
            c->h_trace[1], c->h_trace[2], c->h_trace[3]);
    cudaFreeHost(c->h_trace);
  }
  if (c->h_tline) {
    // per operator: microseconds since the first stamp of the last traced forward
    long long t0 = 0;
    for (int i = 0; i < c->n_ops * 16; ++i) if (c->h_tline[i] && (!t0 || c->h_tline[i] < t0)) t0 = c->h_tline[i];
    fprintf(stderr, "op: epi_in att/pre_sig acc0 epi_out | x_flag x_issued | mma0 | w_issued | tmem_ld partial_done mid_epi after_signal  (us)\n");
    for (int o = 0; o < c->n_ops; ++o) {
      fprintf(stderr, "%3d:", o);
      for (int k = 0; k < 16; ++k) fprintf(stderr, " %8.2f", c->h_tline[o * 16 + k] ? (c->h_tline[o * 16 + k] - t0) / 1000.0 : -1.0);
      fprintf(stderr, "\n");
    }
    cudaFreeHost(c->h_tline);
  }
  delete c;       // the device buffers belong to the handle's slab
  h->mega = nullptr;
}

// Sizes of the persistent kernel's device buffers, in carving order (hot and small first).
struct MegaSizes { size_t sync, model, layers, att_ml, att_o, part, total; int grid; size_t att_slots; };
static MegaSizes mega_sizes(const fdvlm_t* h) {
  const fdvlm_config& cf = h->cfg;
  MegaSizes z;
  memset(&z, 0, sizeof(z));
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  z.grid = sms > 0 ? sms : 1;
  const int d = cf.head_dim, H = cf.hidden, I = cf.intermediate, NQ = cf.n_q_heads * d, NKV = cf.n_kv_heads * d;
  const int tq = ceil_div(NQ, 128) + 2 * ceil_div(NKV, 128), T_o = ceil_div(H, 128), T_g = ceil_div(I, 64), T_l = ceil_div(cf.vocab, 128);
  const int stride = ((C_TILES + tq + T_o + T_g + T_o + 31) / 32) * 32;
  z.sync = ((size_t)cf.n_layers * stride + 32 + T_l + 32) * sizeof(int);
  z.model = sizeof(MgModel);
  z.layers = sizeof(MgLayer) * cf.n_layers;
  size_t worst = 0;
  for (int n = 1; n <= cf.max_block; ++n) {
    // the chunk count of a shorter sequence can exceed that of max_seq (chunks are whole key tiles), so take its bound
    const MgAttPlan p = mg_att_plan(n, cf.max_seq, cf.n_q_heads, cf.n_kv_heads, z.grid);
    int bound = z.grid / (cf.n_kv_heads * p.groups);
    const int tiles_max = ceil_div(cf.max_seq, AT_KEYS);
    if (bound > tiles_max) bound = tiles_max;
    if (bound < 1) bound = 1;
    const size_t slots = (size_t)cf.n_q_heads * n * bound;
    if (slots > worst) worst = slots;
  }
  z.att_slots = worst;
  z.att_ml = worst * sizeof(float2);
  z.att_o = worst * d * sizeof(float);
  z.part = (size_t)z.grid * 2 * 64 * 128 * sizeof(float);
  auto up = [](size_t b) { return (b + 255) / 256 * 256; };
  z.total = up(z.sync) + up(z.model) + up(z.layers) + up(z.att_ml) + up(z.att_o) + up(z.part);
  return z;
}
size_t mega_slab_bytes(const fdvlm_t* h) {
  if (h->dt != DT_BF16) return 16;
  return mega_sizes(h).total;
}

// Builds the device-side model description.  Returns false (and leaves h->mega null) when the shape or the
// device does not fit the persistent kernel; the caller then keeps the kernel-per-operator path.
bool mega_create(fdvlm_t* h) {
  const fdvlm_config& cf = h->cfg;
  h->mega = nullptr;
  if (h->dt != DT_BF16 || !mg_encode_fn()) return false;
  const int d = cf.head_dim, H = cf.hidden, I = cf.intermediate;
  const int NQ = cf.n_q_heads * d, NKV = cf.n_kv_heads * d;
  if ((H % 8) || (I % 16) || (NQ % 8)) return false;
  int dev = 0, coop = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (!coop || sms < 1) return false;

  MegaCtx* c = new MegaCtx;
  c->grid = sms;
  MgModel mt;               // tensor maps (device copy)
  memset(&mt, 0, sizeof(mt));
  MgConst& mm = c->cst;
  memset(&mm, 0, sizeof(mm));
  std::vector<MgLayer> layers(cf.n_layers);
  bool ok = true;
  for (int l = 0; l < cf.n_layers && ok; ++l) {
    const fdvlm_layer_weights& lw = h->layers[l];
    MgLayer& L = layers[l];
    memset(&L, 0, sizeof(L));
    ok = mg_tmap(&L.tm_q, lw.wq, NQ, H, 128) && mg_tmap(&L.tm_k, lw.wk, NKV, H, 128) && mg_tmap(&L.tm_v, lw.wv, NKV, H, 128) &&
         mg_tmap(&L.tm_o, lw.wo, H, NQ, 128) && mg_tmap(&L.tm_d, lw.w_down, H, I, 128) && mg_tmap(&L.tm_g, lw.w_gate, I, H, 16) &&
         mg_tmap(&L.tm_u, lw.w_up, I, H, 16);
    L.bq = lw.bq; L.bk = lw.bk; L.bv = lw.bv; L.g_attn = lw.g_attn; L.g_mlp = lw.g_mlp;
    L.kc = (bf16*)kv_ptr(h, l, 0); L.vc = (bf16*)kv_ptr(h, l, 1);
    L.wq = (const bf16*)lw.wq; L.wk = (const bf16*)lw.wk; L.wv = (const bf16*)lw.wv; L.wo = (const bf16*)lw.wo; L.wd = (const bf16*)lw.w_down;
  }
  const void* table = cf.tie_embeddings ? h->w.embed : h->w.lm_head;
  const int R = cf.max_block;
  ok = ok && mg_tmap(&mt.tm_lm, table, cf.vocab, H, 128);
  if (!ok) { delete c; return false; }

  mm.n_layers = cf.n_layers; mm.H = H; mm.I = I; mm.NQ = NQ; mm.NKV = NKV; mm.hq = cf.n_q_heads; mm.hkv = cf.n_kv_heads;
  mm.R = R; mm.d = d; mm.vocab = cf.vocab; mm.mask_id = cf.mask_id; mm.max_seq = cf.max_seq; mm.nt = h->nt;
  mm.eps = cf.rms_eps; mm.inv_h = 1.f / (float)H; mm.g_final = h->w.g_final;
  mm.h = h->h; mm.xg = (bf16*)h->a; mm.q = (bf16*)h->q; mm.ao = (bf16*)h->ao; mm.act = (bf16*)h->act; mm.ssq = h->ssq;
  mm.cs = (const float2*)h->cs; mm.logits = h->logits; mm.stats = (float4*)h->stats; mm.status = h->info + 3;
  mm.tq_begin[0] = 0; mm.tq_begin[1] = ceil_div(NQ, 128); mm.tq_begin[2] = mm.tq_begin[1] + ceil_div(NKV, 128);
  mm.tq_begin[3] = mm.tq_begin[2] + ceil_div(NKV, 128);
  mm.T_o = ceil_div(H, 128); mm.T_g = ceil_div(I, 64); mm.T_l = ceil_div(cf.vocab, 128);
  mm.KB_h = ceil_div(H, 64); mm.KB_q = ceil_div(NQ, 64); mm.KB_i = ceil_div(I, 64);
  // work partition per operator kind
  {
    const int G = c->grid;
    const int T[5] = {mm.tq_begin[3], mm.T_o, mm.T_g, mm.T_o, mm.T_l};
    const int KB[5] = {mm.KB_h, mm.KB_q, mm.KB_h, mm.KB_i, mm.KB_h};
    for (int k = 0; k < 5; ++k) {
      // QKV / O: few tiles, short K -> a small split whose shares fit the run-ahead ring (the weights are already in
      // shared memory when the activations arrive); D: few tiles, long K -> enough splits to occupy most SMs;
      // gate/up and the LM head: stream-K, every SM streams the same number of bytes.
      int sk = KB[k];
      if (k == OP_QKV || k == OP_O) { sk = (G / 2 + T[k] - 1) / T[k]; if (sk > KB[k] / 4) sk = KB[k] / 4; }
      if (k == OP_D) { sk = (G - G / 8) / T[k]; if (sk > KB[k] / 8) sk = KB[k] / 8; }
      if (sk < 1) sk = 1;
      if (sk > KB[k]) sk = KB[k];
      const long long W = (long long)T[k] * sk;
      mm.op_sk[k] = sk;
      mm.op_ge[k] = W < G ? (int)W : G;
      mm.op_off[k] = (k == OP_O) ? 3 : (k == OP_D ? 5 : 0);
    }
  }
  mm.off_to = C_TILES + mm.tq_begin[3]; mm.off_tg = mm.off_to + mm.T_o; mm.off_td = mm.off_tg + mm.T_g;
  mm.layer_stride = ((mm.off_td + mm.T_o + 31) / 32) * 32;
  mm.off_lm = mm.layer_stride + 32;   // relative to the last layer's counters
  c->sync_bytes = ((size_t)cf.n_layers * mm.layer_stride + 32 + mm.T_l + 32) * sizeof(int);

  const MegaSizes z = mega_sizes(h);
  bool alloc_ok = h->mega_slab != nullptr && z.sync == c->sync_bytes;
  if (alloc_ok) {
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    char* cur = h->mega_slab;
    c->d_sync = (int*)cur; cur += up(z.sync);
    c->d_model = (MgModel*)cur; cur += up(z.model);
    c->d_layers = (MgLayer*)cur; cur += up(z.layers);
    c->d_att_ml = (float2*)cur; cur += up(z.att_ml);
    c->d_att_o = (float*)cur; cur += up(z.att_o);
    c->d_part = (float*)cur;
  }
  const char* tr = getenv("FDVLM_MEGA_TRACE");
  if (alloc_ok && tr && tr[0] == '1' && cudaHostAlloc((void**)&c->h_trace, 64, cudaHostAllocMapped) == cudaSuccess) {
    memset(c->h_trace, 0, 64);
    void* dp = nullptr;
    if (cudaHostGetDevicePointer(&dp, c->h_trace, 0) == cudaSuccess) mm.trace = (int*)dp;
    c->n_ops = cf.n_layers * 4 + 1;
    if (cudaHostAlloc((void**)&c->h_tline, (size_t)c->n_ops * 128, cudaHostAllocMapped) == cudaSuccess) {
      memset(c->h_tline, 0, (size_t)c->n_ops * 128);
      if (cudaHostGetDevicePointer(&dp, c->h_tline, 0) == cudaSuccess) mm.tline = (long long*)dp;
    }
  }
  mm.trace_cta = -1;
  if (mm.tline) { const char* tc = getenv("FDVLM_MEGA_TRACE_CTA"); mm.trace_cta = tc ? atoi(tc) : 0; }
  if (alloc_ok) {
    mm.layers = c->d_layers; mm.sync = c->d_sync; mm.part = c->d_part; mm.att_o = c->d_att_o; mm.att_ml = c->d_att_ml;
    alloc_ok = cudaMemcpy(c->d_layers, layers.data(), sizeof(MgLayer) * cf.n_layers, cudaMemcpyHostToDevice) == cudaSuccess &&
               cudaMemcpy(c->d_model, &mt, sizeof(MgModel), cudaMemcpyHostToDevice) == cudaSuccess;
  }
  h->mega = c;
  if (!alloc_ok) {
    cudaGetLastError();
    mega_destroy(h);
    return false;
  }
  return true;
}

// One forward over the n rows staged in the residual stream (see forward_rows for the arguments).
int mega_forward(fdvlm_t* h, int n, int mode, int logits_rows, int want_logits) {
  MegaCtx* c = (MegaCtx*)h->mega;
  const fdvlm_config& cf = h->cfg;
  launch_rope_table(h->cs, n, h->cache_len, cf.head_dim, cf.rope_theta, h->st);
  CU(h, cudaMemsetAsync(c->d_sync, 0, c->sync_bytes, h->st));
  const MgAttPlan p = mg_att_plan(n, h->cache_len + n, cf.n_q_heads, cf.n_kv_heads, c->grid);
  MgRun run;
  run.M = c->d_model; run.c = c->cst; run.m = n; run.L = h->cache_len; run.causal = (mode == MODE_CAUSAL);
  run.lm_rows = (logits_rows == 0) ? 0 : (logits_rows == n ? n : 1);
  run.write_logits = (logits_rows == n) ? want_logits : 1;
  run.qh = p.qh; run.att_groups = p.groups; run.chunk_keys = p.chunk_keys; run.n_chunks = p.n_chunks;
  prof_begin(h, 0);
  cudaError_t e = (cf.head_dim == 128) ? mg_launch_d<128>(run, c->grid, h->st) : mg_launch_d<64>(run, c->grid, h->st);
  prof_end(h);
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "persistent forward launch: %s", cudaGetErrorString(e));
  h->launches += 2;
  if (logits_rows == n) {
    launch_stats_merge(h->stats, ceil_div(cf.vocab, 128) * 4, n, h->conf, h->pred, h->st);
    h->launches++;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(h, FDVLM_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

}  // namespace fdk
