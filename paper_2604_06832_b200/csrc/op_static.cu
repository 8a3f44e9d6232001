// fdvlm_op_linear_static: the small-M projection of fdvlm_op_linear for callers that must not allocate
// device memory.  Its split-K scratch (and the device word the kernels report a timed-out wait in) lives
// in a file-scope __device__ array that every GPU loading this library holds until the process exits.
#include <mutex>

#include "handle.h"

namespace fdk {
int launch_linear_simt(const LinearArgs& a, cudaStream_t st, cudaError_t* err);
size_t simt_workspace_bytes(int m, int n, int k);
void launch_splitk_epilogue(const float* part, int S, int m, int n, const float* scale, const float* bias, float* y, int ldy,
                            int accumulate, cudaStream_t st);
}  // namespace fdk

using namespace fdk;

// First 256 bytes: the status word; the rest: split-K partial sums.
static __device__ __align__(256) unsigned char g_static_scratch[FDVLM_STATIC_SCRATCH_BYTES];
constexpr size_t STATIC_HEAD = 256;
constexpr int MAX_DEVICES = 64;

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
  const bool tc = tc_linear_supported(m, n, k, (int)dtype);
  const size_t need = tc ? tc_workspace_bytes(m, n, (n + 127) / 128, k) : simt_workspace_bytes(m, n, k);
  const size_t room = (size_t)FDVLM_STATIC_SCRATCH_BYTES - STATIC_HEAD;
  if (need > room)
    return fail(nullptr, FDVLM_ERR_CAPACITY,
                "op_linear_static: m=%d n=%d k=%d needs %zu bytes of split-K scratch, the built-in scratch holds %zu; "
                "use fdvlm_op_linear with a caller-provided workspace",
                m, n, k, need, room);
  cudaError_t e = cudaSuccess;
  unsigned char* base = static_scratch_of_current_device(&e);
  if (!base) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  float* part = (float*)(base + STATIC_HEAD);
  if (!tc) {
    LinearArgs a;
    a.x = x; a.w = w; a.scale = scale; a.bias = bias; a.y = y; a.m = m; a.n = n; a.k = k; a.ldy = n; a.accumulate = 0;
    a.dtype = (int)dtype; a.workspace = part; a.workspace_bytes = room;
    return launch_linear_simt(a, st, &e) < 0 ? fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: %s", cudaGetErrorString(e))
                                             : (int)FDVLM_OK;
  }
  // the status word must read zero when the kernel starts (an earlier call may have left a report there);
  // the partial sums need no clearing: every (tile, split) slot that is summed is written by this call
  e = cudaMemsetAsync(base, 0, sizeof(int), st);
  if (e != cudaSuccess) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
  TcGroup g;
  memset(&g, 0, sizeof(g));
  g.x = x; g.m = m; g.k = k; g.w[0] = w; g.n[0] = n; g.n_mats = 1;
  g.fp8 = (dtype == FDVLM_W_FP8E4M3);
  int splits = 0;
  TcOut o;
  memset(&o, 0, sizeof(o));
  o.mode = TC_MODE_PARTIAL; o.part = part; o.part_bytes = room; o.splits_out = &splits; o.ld = n; o.status = (int*)base;
  e = tc_group_launch(g, o, st);
  if (e != cudaSuccess) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: GEMM launch: %s", cudaGetErrorString(e));
  launch_splitk_epilogue(part, splits, m, n, scale, bias, y, n, 0, st);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, FDVLM_ERR_CUDA, "op_linear_static: reduce launch: %s", cudaGetErrorString(e));
  return FDVLM_OK;
}
