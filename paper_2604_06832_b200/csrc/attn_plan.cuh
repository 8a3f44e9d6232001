// What the two attention kernels (mma.sync and tcgen05) and their chunk-merge kernel share.
#pragma once
#include "common.cuh"

namespace fdk {

constexpr int AT_KEYS = 64;    // keys per shared-memory tile
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Split of T keys into chunks of whole 64-key tiles, at most `bound` chunks (the same on host and device, so a launch
// whose grid was sized for `bound` can take the sequence length from device memory).
__host__ __device__ inline void attn_chunking(int T, int bound, int* chunk_keys, int* n_chunks) {
  const int tiles = (T + AT_KEYS - 1) / AT_KEYS;
  int want = bound < tiles ? bound : tiles;
  if (want < 1) want = 1;
  *chunk_keys = ((tiles + want - 1) / want) * AT_KEYS;
  *n_chunks = (T + *chunk_keys - 1) / *chunk_keys;
}


}  // namespace fdk
