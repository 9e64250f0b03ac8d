// Status strings, device-status read-back and the launch counter.
#include <cstdlib>

#include "common.cuh"

namespace ss {
std::atomic<long long> g_launch_count{0};

bool pdl_enabled() {
  static const bool on = std::getenv("SS_NO_PDL") == nullptr;
  return on;
}
}

extern "C" const char* ss_status_string(int32_t status) {
  switch (status) {
    case SS_OK: return "ok";
    case SS_ERR_INVALID_ARG: return "invalid argument";
    case SS_ERR_UNSUPPORTED: return "unsupported shape or layout";
    case SS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SS_ERR_CUDA: return "CUDA call failed";
    case SS_ERR_BAD_INPUT: return "index out of range in a descriptor array";
    case SS_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown status";
  }
}

extern "C" int32_t ss_last_device_status(const void* workspace, void* stream, int32_t* out_status) {
  if (!workspace || !out_status) return SS_ERR_INVALID_ARG;
  cudaStream_t st = ss::as_stream(stream);
  if (cudaMemcpyAsync(out_status, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  if (cudaStreamSynchronize(st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  return SS_OK;
}

extern "C" int64_t ss_launch_count(void) { return ss::g_launch_count.load(std::memory_order_relaxed); }
