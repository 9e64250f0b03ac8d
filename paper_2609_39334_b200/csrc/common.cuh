// Shared host/device helpers of the specscale CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>
#include <stddef.h>

#include "../../include/specscale.h"

namespace ss {

// Host-side count of kernel launches made by this library (diagnostic, see ss_launch_count).
extern std::atomic<long long> g_launch_count;   // (atomic: hosts may call from one thread per stream)

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// True unless the environment variable SS_NO_PDL is set (read once): launch kernels with programmatic stream
// serialization, i.e. let a kernel's blocks become resident while the kernel before it on the stream is still
// draining.  Every kernel of the library starts with grid_dependency_enter(), which does not return before the
// preceding kernel has completed and its writes are visible, so the results are those of plain stream order; what
// is saved is the launch latency between dependent kernels (several microseconds each, most of a small step).
bool pdl_enabled();

// Every kernel launch in the library goes through this macro so that launches are counted and launch errors
// are turned into SS_ERR_CUDA.
#define SS_LAUNCH(kernel, grid_, block_, smem_, stream_, ...)                         \
  do {                                                                            \
    cudaLaunchConfig_t ss_cfg_ = {};                                              \
    ss_cfg_.gridDim = dim3(static_cast<unsigned>(grid_));                          \
    ss_cfg_.blockDim = dim3(static_cast<unsigned>(block_));                        \
    ss_cfg_.dynamicSmemBytes = static_cast<size_t>(smem_);                        \
    ss_cfg_.stream = (stream_);                                                   \
    cudaLaunchAttribute ss_attr_[1];                                              \
    ss_attr_[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;          \
    ss_attr_[0].val.programmaticStreamSerializationAllowed = 1;                   \
    ss_cfg_.attrs = ss_attr_;                                                     \
    ss_cfg_.numAttrs = ::ss::pdl_enabled() ? 1 : 0;                               \
    const cudaError_t ss_err_ = cudaLaunchKernelEx(&ss_cfg_, kernel, __VA_ARGS__); \
    ::ss::g_launch_count.fetch_add(1, std::memory_order_relaxed);                 \
    if (ss_err_ != cudaSuccess || cudaPeekAtLastError() != cudaSuccess) {         \
      (void)cudaGetLastError();                                                   \
      return SS_ERR_CUDA;                                                         \
    }                                                                             \
  } while (0)

// Function attributes and device properties are per device, so "done once" caches are arrays indexed by the current
// device.  Returns the device's index, or -1 when it cannot be used as an index (the caller then skips its cache).
// The host-side caches of the library (these, the launch counter, the event profiler) are not guarded by locks:
// calls that share a device must come from one thread at a time.
constexpr int kDeviceSlots = 64;
inline int current_device_slot() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return -1; }
  return (dev >= 0 && dev < kDeviceSlots) ? dev : -1;
}

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
// First statement of every kernel (see pdl_enabled): allow the next kernel on the stream to be scheduled early, then
// wait until the previous kernel has completed and flushed its writes.  Both are no-ops for a kernel launched
// without the programmatic-serialization attribute.  It must run unconditionally: a kernel that exited without
// waiting could complete before its predecessor, and its successor would then start too early.
__device__ __forceinline__ void grid_dependency_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Two variants for a pair of kernels that may overlap.  The EARLIER kernel of the pair enters with
// grid_dependency_enter_then_release(): it waits for its own predecessor first and only then lets its successor be
// scheduled, so the successor's blocks cannot start before that predecessor's results are complete.  The LATER kernel
// enters with grid_dependency_release() alone, works on what does not depend on the earlier kernel, and calls
// grid_dependency_wait() before it first touches the earlier kernel's results - and, in every thread, before it
// exits, so that the kernel after it still sees plain stream order.
__device__ __forceinline__ void grid_dependency_enter_then_release() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
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

// Checked build (-DSS_CHECKED, libspecscale_checked.so): range predicates on the kernels' OWN address arithmetic - page
// ids against the pool, partial slots against the workspace capacity, query / output rows against the tensors.  A
// failed predicate records SS_ERR_BAD_INPUT in the status word and runs `fallback` (clamp the index or skip the
// access), so nothing is ever accessed out of range.  In the production build the macro expands to nothing.
#ifdef SS_CHECKED
#define SS_CHECK_OR(cond, status_ptr, fallback)                         \
  do {                                                                  \
    if (!(cond)) {                                                      \
      ::ss::set_status((status_ptr), SS_ERR_BAD_INPUT);                 \
      fallback;                                                         \
    }                                                                   \
  } while (0)
#else
#define SS_CHECK_OR(cond, status_ptr, fallback) do { } while (0)
#endif
#endif

}  // namespace ss
