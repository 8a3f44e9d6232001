// Shared device/host helpers of the fdvlm CUDA library (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

namespace fdk {

typedef __nv_bfloat16 bf16;
struct fp8e4m3 { uint8_t b; };  // OCP e4m3fn storage byte

// ---- exact widening of storage types to fp32 -------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
// e4m3 (1-4-3, bias 7) placed in a half (1-5-10, bias 15): same sign, exponent field and top
// mantissa bits; the bias difference is a factor 2^8.  Exact for normals and subnormals alike.
__device__ __forceinline__ float to_f32(fp8e4m3 v) {
  unsigned short hb = (unsigned short)(((v.b & 0x80u) << 8) | ((v.b & 0x7Fu) << 7));
  return __half2float(__ushort_as_half(hb)) * 256.0f;
}

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) {
  unsigned short r;
  asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(r) : "f"(v));
  return __ushort_as_half(r);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum / max through shared memory (blockDim.x a multiple of 32, <= 1024).
__device__ __forceinline__ float block_sum(float v, float* red) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float r = (lane < nw) ? red[lane] : 0.f;
  r = warp_sum(r);
  return r;
}
__device__ __forceinline__ float block_max(float v, float* red) {
  int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float r = (lane < nw) ? red[lane] : -INFINITY;
  r = warp_max(r);
  return r;
}

// Programmatic dependent launch: a kernel launched with launch_pdl may start while its predecessor in the stream is
// still running.  pdl_trigger lets the successor's CTAs be scheduled early; pdl_wait returns once the predecessor grid
// has completed and its writes are visible -- every thread calls it before it reads the predecessor's results or
// overwrites anything the predecessor may still read.  Launched the ordinary way both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Set while a launch sequence is captured for a place that takes no programmatic edges: the kernels are then launched
// the ordinary way (pdl_trigger / pdl_wait are no-ops).
inline bool& pdl_disabled() {
  static thread_local bool off = false;
  return off;
}
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl_disabled() ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// In-chain timing of one kernel launch (only when profiling is on; a null pointer otherwise): the earliest start of
// any of its CTAs, the earliest return of any CTA from its wait for the predecessor grid, the latest end of any CTA,
// all in nanoseconds of the GPU's global timer.  Every field is kept as a minimum (the end as the minimum of the
// complemented time), so the host presets the whole record to all-ones bytes.
struct KStamp { unsigned long long start, released, end_inv, pad; };
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Each called by ONE thread of a CTA.  A CTA that can see it would not lower the minimum skips the atomic (hundreds of
// CTAs updating one word would stretch the small kernels they are meant to time); `sampled` end stamps, for kernels of
// many short equal CTAs, come from every eighth CTA and the last one only.
__device__ __forceinline__ void stamp_min(unsigned long long* p, unsigned long long t) {
  if (t < *reinterpret_cast<volatile unsigned long long*>(p)) atomicMin(p, t);
}
__device__ __forceinline__ void stamp_start(KStamp* s) { if (s) stamp_min(&s->start, global_ns()); }
__device__ __forceinline__ void stamp_released(KStamp* s) { if (s) stamp_min(&s->released, global_ns()); }
__device__ __forceinline__ void stamp_end(KStamp* s, bool sampled = false) {
  if (!s) return;
  if (sampled) {
    const unsigned id = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
    const unsigned total = gridDim.x * gridDim.y * gridDim.z;
    if ((id & 7u) != 0 && id != total - 1) return;
  }
  atomicMin(&s->end_inv, ~global_ns());
}

// MASKED: per-row bit masks among the rows + per-row position ids (Appendix B, Alg. 2).  FUSED: the causal commit of a
// finished block and the first denoise step of the next block as one forward (per-row bit masks, natural positions).
enum { MODE_BIDIR = 0, MODE_CAUSAL = 1, MODE_MASKED = 2, MODE_FUSED = 3 };
enum { DT_F32 = 0, DT_BF16 = 1, DT_FP8 = 2, DT_A8 = 3 };   // DT_A8: fp8 weights and per-row fp8 inputs (stand-alone projection only)
// Element type of q and the KV cache on the tensor-core path.
enum { KV_BF16 = 0, KV_F16 = 1 };
// How a 16-bit activation tensor that feeds a tensor-core GEMM is stored.
//   XF_BF16X2: two bf16 planes, hi = bf16(v) and lo = bf16(v - hi), `lo_off` elements apart: the GEMM multiplies
//              the streamed weight tile by both, so the activation carries ~16 significant bits (bf16 weights).
//   XF_F16   : one f16 plane (fp8 weights widen exactly to f16, so that GEMM runs in f16: 11 significant bits).
//   XF_BF16  : one bf16 plane (operator-level entry points that take caller-given bf16 rows).
enum { XF_BF16X2 = 0, XF_F16 = 1, XF_BF16 = 2 };
// Device status word: 0 = fine; 1..15 = a bounded wait gave up (the role that gave up); 16 = a token id outside
// [0, vocab) was met (row 0 of the table was read instead).
enum { ST_PRODUCER = 1, ST_MMA = 2, ST_EPILOGUE = 3, ST_ATTENTION = 4, ST_BAD_TOKEN = 16 };

__device__ __forceinline__ unsigned short f16_bits_sat(float v) {
  unsigned short r;
  asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(r) : "f"(v));
  return r;
}
// one activation value into a tensor stored as `fmt` (see above); p points at the hi / only plane
__device__ __forceinline__ void store_act(void* p, size_t lo_off, size_t idx, float v, int fmt) {
  if (fmt == XF_F16) {
    reinterpret_cast<unsigned short*>(p)[idx] = f16_bits_sat(v);
  } else {
    const bf16 hi = __float2bfloat16_rn(v);
    reinterpret_cast<bf16*>(p)[idx] = hi;
    if (fmt == XF_BF16X2) reinterpret_cast<bf16*>(p)[lo_off + idx] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

constexpr int MAX_DEVICES = 64;
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) is a per-device setting: `done` is one flag per device.
template <typename K>
static inline cudaError_t ensure_dynamic_smem(K kern, int bytes, bool* done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done[dev] = true;
  return e;
}

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace fdk
