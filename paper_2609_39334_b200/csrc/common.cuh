// Shared host/device helpers of the specscale CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/specscale.h"

namespace ss {

// Host-side count of kernel launches made by this library (diagnostic, see ss_launch_count).
extern long long g_launch_count;

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// Every kernel launch in the library goes through this macro so that launches are counted and launch errors
// are turned into SS_ERR_CUDA.
#define SS_LAUNCH(kernel, grid, block, smem, stream, ...)                         \
  do {                                                                            \
    kernel<<<(grid), (block), (smem), (stream)>>>(__VA_ARGS__);                   \
    ++::ss::g_launch_count;                                                       \
    if (cudaPeekAtLastError() != cudaSuccess) { (void)cudaGetLastError(); return SS_ERR_CUDA; } \
  } while (0)

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Carves aligned regions out of a caller workspace (host-side bookkeeping only).
struct Carver {
  char* base;
  size_t off;
  explicit Carver(void* p) : base(static_cast<char*>(p)), off(0) {}
  template <typename T>
  T* take(size_t count) {
    T* p = reinterpret_cast<T*>(base + off);
    off = align_up(off + count * sizeof(T));
    return p;
  }
};

__host__ __device__ inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

#ifdef __CUDACC__
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
// First error wins: the status word keeps the first non-zero code written to it.
__device__ __forceinline__ void set_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }
#endif

}  // namespace ss
