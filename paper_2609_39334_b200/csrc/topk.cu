// ss_topk_prune: keep the k best-scored candidates of every problem (paper, Section "Early Pruning of Search
// Tree": a candidate ranked below the top-k cannot be selected; Section "Test-Time Scaling": k = N / M).
//
// One block per segment.  Each candidate becomes a 64-bit key (order-reversed score bits << 32 | local
// index), so ascending key order is "score descending, index ascending" and all keys are distinct; the block
// sorts the keys with a bitonic network in shared memory (segments up to kSmemKeys candidates) or in the
// caller's workspace (larger segments), then writes the first k indices and the keep mask.
#include "common.cuh"

namespace ss {
namespace topk {

constexpr int kThreads = 256;
constexpr int kSmemKeys = 4096;     // 32 KB of shared memory

__device__ __forceinline__ uint64_t make_key(float f, uint32_t local_idx) {
  uint32_t ordered;                           // ascending in the score
  if (f != f) {
    ordered = 0u;                             // NaN below every number (below -inf, whose code is 0x007fffff)
  } else {
    f = f + 0.0f;                             // -0.0 -> +0.0
    const uint32_t u = __float_as_uint(f);
    ordered = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  }
  return (static_cast<uint64_t>(~ordered) << 32) | local_idx;
}

__device__ void bitonic_sort(uint64_t* keys, int n_pad) {
  for (int size = 2; size <= n_pad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = threadIdx.x; t < (n_pad >> 1); t += blockDim.x) {
        const int lo = ((t / stride) * (stride << 1)) + (t % stride);
        const int hi = lo + stride;
        const bool up = ((lo & size) == 0);
        const uint64_t a = keys[lo], b = keys[hi];
        if ((a > b) == up) { keys[lo] = b; keys[hi] = a; }
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(kThreads)
topk_kernel(const float* __restrict__ scores, const int32_t* __restrict__ seg_offsets, int n_total, int k,
            int32_t* __restrict__ survivors, uint8_t* __restrict__ keep, uint64_t* __restrict__ scratch,
            int32_t* __restrict__ status) {
  ss::grid_dependency_enter();
  __shared__ uint64_t smem_keys[kSmemKeys];
  const int s = blockIdx.x;
  const int lo = seg_offsets[s], hi = seg_offsets[s + 1];
  // a segment that does not lie inside [0, n_total] is reported and treated as empty: its offsets index keep[] and
  // the scratch region, so following them would write out of bounds
  const bool bad = lo < 0 || hi < lo || hi > n_total;
  if (bad && threadIdx.x == 0) set_status(status, SS_ERR_BAD_INPUT);
  const int n = bad ? 0 : hi - lo;
  if (n <= 0) {
    for (int j = threadIdx.x; j < k; j += blockDim.x) survivors[static_cast<int64_t>(s) * k + j] = -1;
    return;
  }
  int n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  // A segment's scratch region starts at 2*lo: pow2ceil(n) < 2n keeps the regions of different segments apart.
  uint64_t* keys = (n_pad <= kSmemKeys) ? smem_keys : (scratch + 2 * static_cast<int64_t>(lo));
  for (int i = threadIdx.x; i < n_pad; i += blockDim.x)
    keys[i] = i < n ? make_key(scores[lo + i], static_cast<uint32_t>(i)) : ~0ull;
  __syncthreads();
  bitonic_sort(keys, n_pad);
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const int cand = lo + static_cast<int>(keys[j] & 0xffffffffu);
    keep[cand] = j < k ? 1 : 0;
    if (j < k) survivors[static_cast<int64_t>(s) * k + j] = cand;
  }
  for (int j = n + threadIdx.x; j < k; j += blockDim.x) survivors[static_cast<int64_t>(s) * k + j] = -1;
}

// Early pruning with partially verified candidates (paper, Section "Early Pruning of Search Tree").  Same sort as
// above over the VERIFIED candidates only (the others get the padding key and sort last); then
//   rule 2: >= k verified candidates with the perfect score  -> the first k of them by index are selected, every
//           other candidate of the segment is pruned, the segment is final;
//   rule 1: more than k verified -> the verified candidates ranked below the k best are pruned;
//   all verified -> final, selected = the k best.
__global__ void __launch_bounds__(kThreads)
early_prune_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ verified,
                   const int32_t* __restrict__ seg_offsets, int n_total, int k, uint8_t* __restrict__ pruned,
                   int32_t* __restrict__ selected, uint8_t* __restrict__ final_out, uint64_t* __restrict__ scratch,
                   int32_t* __restrict__ status) {
  ss::grid_dependency_enter();
  __shared__ uint64_t smem_keys[kSmemKeys];
  __shared__ int s_nver, s_nperfect;
  const int s = blockIdx.x;
  const int lo = seg_offsets[s], hi = seg_offsets[s + 1];
  const bool bad = lo < 0 || hi < lo || hi > n_total;        // (see topk_kernel)
  if (bad && threadIdx.x == 0) set_status(status, SS_ERR_BAD_INPUT);
  const int n = bad ? 0 : hi - lo;
  for (int j = threadIdx.x; j < k; j += blockDim.x) selected[static_cast<int64_t>(s) * k + j] = -1;
  if (n <= 0) {
    if (threadIdx.x == 0) final_out[s] = 1;      // nothing left to verify in an empty segment
    return;
  }
  if (threadIdx.x == 0) { s_nver = 0; s_nperfect = 0; }
  __syncthreads();
  int n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  uint64_t* keys = (n_pad <= kSmemKeys) ? smem_keys : (scratch + 2 * static_cast<int64_t>(lo));
  int my_ver = 0, my_perfect = 0;
  for (int i = threadIdx.x; i < n_pad; i += blockDim.x) {
    uint64_t key = ~0ull;
    if (i < n && verified[lo + i]) {
      const float f = scores[lo + i];
      key = make_key(f, static_cast<uint32_t>(i));
      ++my_ver;
      if (f >= 1.0f) ++my_perfect;
    }
    keys[i] = key;
  }
  if (my_ver) atomicAdd(&s_nver, my_ver);
  if (my_perfect) atomicAdd(&s_nperfect, my_perfect);
  __syncthreads();
  const int nver = s_nver, nperfect = s_nperfect;
  if (nperfect >= k) {
    // rule 2: rank of a perfect candidate among the perfect ones by index (segments are small: a counting loop)
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      bool chosen = false;
      if (verified[lo + i] && scores[lo + i] >= 1.0f) {
        int before = 0;
        for (int j = 0; j < i; ++j) before += (verified[lo + j] && scores[lo + j] >= 1.0f) ? 1 : 0;
        if (before < k) {
          chosen = true;
          selected[static_cast<int64_t>(s) * k + before] = lo + i;
        }
      }
      pruned[lo + i] = chosen ? 0 : 1;
    }
    if (threadIdx.x == 0) final_out[s] = 1;
    return;
  }
  bitonic_sort(keys, n_pad);
  const bool all_verified = nver == n;
  for (int i = threadIdx.x; i < n; i += blockDim.x)
    if (!verified[lo + i]) pruned[lo + i] = 0;
  for (int j = threadIdx.x; j < nver; j += blockDim.x) {
    const int cand = lo + static_cast<int>(keys[j] & 0xffffffffu);
    pruned[cand] = (nver > k && j >= k) ? 1 : 0;
    if (all_verified && j < k) selected[static_cast<int64_t>(s) * k + j] = cand;
  }
  if (threadIdx.x == 0) final_out[s] = all_verified ? 1 : 0;
}

}  // namespace topk
}  // namespace ss

extern "C" int32_t ss_early_prune(const float* scores, const uint8_t* verified, const int32_t* seg_offsets,
                                  int32_t n_segments, int32_t n_total, int32_t k, uint8_t* pruned_out,
                                  int32_t* selected_out, uint8_t* final_out, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  using namespace ss;
  if (n_segments < 0 || n_total < 0 || k < 1) return SS_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (n_total > 0 && pruned_out && cudaMemsetAsync(pruned_out, 0, static_cast<size_t>(n_total), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  if (n_segments == 0) return SS_OK;
  if (!seg_offsets || !selected_out || !final_out || !workspace) return SS_ERR_INVALID_ARG;
  if (n_total > 0 && (!scores || !verified || !pruned_out)) return SS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return SS_ERR_INVALID_ARG;
  size_t need = 0;
  ss_topk_workspace_bytes(n_total, &need);
  if (workspace_bytes < need) return SS_ERR_WORKSPACE_TOO_SMALL;
  if (cudaMemsetAsync(workspace, 0, sizeof(int32_t), st) != cudaSuccess) { (void)cudaGetLastError(); return SS_ERR_CUDA; }
  SS_LAUNCH(topk::early_prune_kernel, n_segments, topk::kThreads, 0, st, scores, verified, seg_offsets, n_total, k,
            pruned_out, selected_out, final_out, reinterpret_cast<uint64_t*>(static_cast<char*>(workspace) + kAlign),
            static_cast<int32_t*>(workspace));
  return SS_OK;
}

extern "C" int32_t ss_topk_workspace_bytes(int32_t n_total, size_t* out_bytes) {
  if (n_total < 0 || !out_bytes) return SS_ERR_INVALID_ARG;
  // the status word (first bytes, see ss_last_device_status), then two 64-bit sort keys per candidate
  *out_bytes = ss::kAlign + ss::align_up(static_cast<size_t>(2) * (n_total > 0 ? n_total : 1) * sizeof(uint64_t));
  return SS_OK;
}

extern "C" int32_t ss_topk_prune(const float* scores, const int32_t* seg_offsets, int32_t n_segments,
                                 int32_t n_total, int32_t k, int32_t* survivors_out, uint8_t* keep_out,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  using namespace ss;
  if (n_segments < 0 || n_total < 0 || k < 1) return SS_ERR_INVALID_ARG;
  if (n_segments == 0) {
    if (n_total > 0 && keep_out &&
        cudaMemsetAsync(keep_out, 0, static_cast<size_t>(n_total), as_stream(stream)) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    return SS_OK;
  }
  if (!seg_offsets || !survivors_out || !workspace) return SS_ERR_INVALID_ARG;
  if (n_total > 0 && (!scores || !keep_out)) return SS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return SS_ERR_INVALID_ARG;
  size_t need = 0;
  ss_topk_workspace_bytes(n_total, &need);
  if (workspace_bytes < need) return SS_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = as_stream(stream);
  if (n_total > 0 && cudaMemsetAsync(keep_out, 0, static_cast<size_t>(n_total), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  if (cudaMemsetAsync(workspace, 0, sizeof(int32_t), st) != cudaSuccess) { (void)cudaGetLastError(); return SS_ERR_CUDA; }
  SS_LAUNCH(topk::topk_kernel, n_segments, topk::kThreads, 0, st, scores, seg_offsets, n_total, k, survivors_out, keep_out,
            reinterpret_cast<uint64_t*>(static_cast<char*>(workspace) + kAlign), static_cast<int32_t*>(workspace));
  return SS_OK;
}
