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
// e4m3 (1-4-3, bias 7) placed in a half (1-5-10, bias 15): same sign, exponent field and top
// mantissa bits; the bias difference is a factor 2^8.  Exact for normals and subnormals alike.
__device__ __forceinline__ float to_f32(fp8e4m3 v) {
  unsigned short hb = (unsigned short)(((v.b & 0x80u) << 8) | ((v.b & 0x7Fu) << 7));
  return __half2float(__ushort_as_half(hb)) * 256.0f;
}

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

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

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

enum { MODE_BIDIR = 0, MODE_CAUSAL = 1 };
enum { DT_F32 = 0, DT_BF16 = 1, DT_FP8 = 2 };

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace fdk
