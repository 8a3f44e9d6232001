// fdvlm_op_linear_static: the small-M projection of fdvlm_op_linear for callers that must not allocate
// device memory.  Its split-K scratch (and the device word the kernels report a timed-out wait in) lives
// in a file-scope __device__ array that every GPU loading this library holds until the process exits.
#include <mutex>

#include "handle.h"

using namespace fdk;

// Laid out like the workspace of fdvlm_op_linear: the status words first, then the kernels' scratch.
static __device__ __align__(256) unsigned char g_static_scratch[FDVLM_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the address a
// kernel may use comes from cudaGetSymbolAddress, asked once per device with that device current.
static unsigned char* static_scratch_of_current_device(cudaError_t* err) {
  static unsigned char* ptrs[MAX_DEVICES] = {};
  static std::mutex mu;
  int dev = -1;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= MAX_DEVICES) { *err = cudaErrorInvalidDevice; return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  if (!ptrs[dev]) {
    void* p = nullptr;
    *err = cudaGetSymbolAddress(&p, g_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    ptrs[dev] = (unsigned char*)p;
  }
  return ptrs[dev];
}

extern "C" int fdvlm_op_linear_static(const void* x, const void* w, const float* scale, const float* bias, float* y, int m,
                                      int n, int k, fdvlm_dtype dtype, void* cuda_stream) {
  if (!x || !w || !y || m < 1 || m > 64 || n < 1 || k < 8 || (k % 8))
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "op_linear_static: NULL pointer or m/n/k out of range");
  if (dtype != FDVLM_F32 && dtype != FDVLM_BF16 && dtype != FDVLM_W_FP8E4M3)
    return fail(nullptr, FDVLM_ERR_INVALID_ARG, "op_linear_static: unknown dtype %d", (int)dtype);
  if (dtype == FDVLM_W_FP8E4M3 && !scale) return fail(nullptr, FDVLM_ERR_INVALID_ARG, "op_linear_static: fp8 weights need scales");
  const size_t need = linear_workspace_bytes(m, n, k, (int)dtype);
  const size_t room = (size_t)FDVLM_STATIC_SCRATCH_BYTES;
  if (need > room)
    return fail(nullptr, FDVLM_ERR_CAPACITY,
                "op_linear_static: m=%d n=%d k=%d needs %zu bytes of scratch, the built-in scratch holds %zu; "
                "use fdvlm_op_linear with a caller-provided workspace",
                m, n, k, need, room);
  cudaError_t e = cudaSuccess;
  unsigned char* base = static_scratch_of_current_device(&e);
  if (!base) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
  // The status words are cleared on the stream by the launcher (an earlier call may have left a report there); the
  // partial sums need no clearing: every (tile, split) slot that is summed is written by this call.
  LinearArgs a;
  a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = n; a.k = k; a.ldy = n; a.accumulate = 0;
  a.dtype = (int)dtype; a.workspace = base; a.workspace_bytes = room;
  if (launch_linear(a, (cudaStream_t)cuda_stream, &e) < 0)
    return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}

extern "C" int fdvlm_op_linear_status(const void* workspace, void* cuda_stream) {
  cudaError_t e = cudaSuccess;
  const void* words = workspace ? workspace : static_scratch_of_current_device(&e);
  if (!words) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_status: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
  int code = 0;
  e = cudaMemcpyAsync(&code, words, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_status: %s", cudaGetErrorString(e));
  if (code != 0)
    return fail(nullptr, FDVLM_ERR_TIMEOUT, "a bounded device-side wait of the projection gave up (kernel role %d); its output is invalid", code);
  return FDVLM_OK;
}
