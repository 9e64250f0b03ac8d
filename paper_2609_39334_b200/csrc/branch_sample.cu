// ss_branch_sample: the sampling half of on-demand branching (paper, Section "Computation Deduplication"): a
// sequence with potential size n draws n next tokens as independent trials from ONE logits row; equal draws are
// grouped afterwards with ss_dedup_paths on (sequence, token) pairs.
//
// One block per sequence.  The cost is the fp64 exponentials (the token decision is taken in fp64 so that it agrees
// with a plain fp64 CPU evaluation except for draws within ~1e-15 of a boundary), so they are evaluated once per
// logit where possible:
//   1. maximum                                   (fp32, exact; the row then stays in L2)
//   2. running sum of exp((logit_v - max) / T) in chunks of 4096 tokens (fp64, block scan): only the cumulative sum
//      at the end of every chunk is kept; the last one is the normaliser Z
//   3. every draw finds its chunk by binary search over those sums; the chunks that hold a draw (one or two for a
//      typical potential size) are evaluated again, now keeping the whole CDF in shared memory, and the draw finds
//      its token by binary search there.
// Bound by the fp64 pipe, not by memory: about one fp64 exponential per logit instead of two.
#include "common.cuh"

namespace ss {
namespace sample {

constexpr int kThreads = 1024;
constexpr int kPerThread = 4;
constexpr int kChunk = kThreads * kPerThread;
constexpr int kMaxChunks = 512;                              // vocabularies of up to 2 M tokens

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kThreads)
branch_sample_kernel(const float* __restrict__ logits, const int64_t* __restrict__ draw_offsets,
                     const float* __restrict__ uniforms, int vocab, double inv_temperature,
                     int32_t* __restrict__ tokens_out, int64_t* __restrict__ seq_out) {
  ss::grid_dependency_enter();
  __shared__ double s_cdf[kChunk];
  __shared__ double s_warp[32];
  __shared__ float s_wmax[32];
  __shared__ double s_end[kMaxChunks];                     // cumulative sum at the end of every chunk
  __shared__ int s_need[kMaxChunks];
  const int s = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* row = logits + static_cast<int64_t>(s) * vocab;
  const int64_t d0 = draw_offsets[s], d1 = draw_offsets[s + 1];
  if (d1 <= d0) return;                                      // nothing to draw for this sequence

  // ---- 1. maximum ---------------------------------------------------------------------------------------------
  float mx = -INFINITY;
  for (int v = tid; v < vocab; v += kThreads) mx = fmaxf(mx, row[v]);
  mx = warp_max(mx);
  if (lane == 0) s_wmax[warp] = mx;
  __syncthreads();
  mx = s_wmax[0];
#pragma unroll
  for (int w = 1; w < 32; ++w) mx = fmaxf(mx, s_wmax[w]);
  const double dmax = static_cast<double>(mx);

  // ---- 2. cumulative sums at the chunk ends; Z -----------------------------------------------------------------------
  // inclusive CDF of chunk `base`: thread t owns tokens base + 4t .. base + 4t + 3; returns the chunk's last value and,
  // if `keep`, leaves every value in s_cdf
  auto chunk_cdf = [&](int base, double carry, bool keep) -> double {
    double e[kPerThread], run = 0.0;
#pragma unroll
    for (int x = 0; x < kPerThread; ++x) {
      const int v = base + tid * kPerThread + x;
      e[x] = v < vocab ? exp((static_cast<double>(row[v]) - dmax) * inv_temperature) : 0.0;
      run += e[x];
    }
    double incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    __syncthreads();                                         // (s_warp / s_cdf of the previous chunk are no longer read)
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      double t = s_warp[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const double y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      s_warp[lane] = t;
    }
    __syncthreads();
    double c = carry + (warp ? s_warp[warp - 1] : 0.0) + incl - run;
    if (keep) {
#pragma unroll
      for (int x = 0; x < kPerThread; ++x) {
        c += e[x];
        s_cdf[tid * kPerThread + x] = c;
      }
      __syncthreads();
    }
    return carry + s_warp[31];
  };
  const int n_chunks = (vocab + kChunk - 1) / kChunk;
  {
    double carry = 0.0;
    for (int k = 0; k < n_chunks; ++k) {
      carry = chunk_cdf(k * kChunk, carry, false);
      if (tid == 0) s_end[k] = carry;
    }
  }
  __syncthreads();
  const double Z = s_end[n_chunks - 1];

  // ---- 3. the draws, in batches of one per thread ----------------------------------------------------------------------
  for (int64_t db = d0; db < d1; db += kThreads) {
    const int64_t d = db + tid;
    const bool have = d < d1;
    const double target = have ? static_cast<double>(uniforms[d]) * Z : 0.0;
    int token = vocab - 1;                                   // the answer if rounding leaves the target above the total
    int my_chunk = -1;
    if (have && s_end[n_chunks - 1] > target) {              // first chunk whose end exceeds the target
      int lo = 0, hi = n_chunks - 1;
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_end[mid] > target) hi = mid; else lo = mid + 1;
      }
      my_chunk = lo;
    }
    for (int k = tid; k < n_chunks; k += kThreads) s_need[k] = 0;
    __syncthreads();
    if (my_chunk >= 0) s_need[my_chunk] = 1;
    __syncthreads();
    for (int k = 0; k < n_chunks; ++k) {
      if (!s_need[k]) continue;                              // (block-uniform)
      chunk_cdf(k * kChunk, k ? s_end[k - 1] : 0.0, true);
      if (my_chunk == k) {                                   // first index of the chunk whose CDF exceeds the target
        int lo = 0, hi = min(kChunk, vocab - k * kChunk) - 1;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (s_cdf[mid] > target) hi = mid; else lo = mid + 1;
        }
        token = k * kChunk + lo;
      }
    }
    if (have) {
      tokens_out[d] = token;
      seq_out[d] = s;
    }
    __syncthreads();
  }
}

}  // namespace sample
}  // namespace ss

extern "C" int32_t ss_branch_sample(const float* logits, const int64_t* draw_offsets, const float* uniforms,
                                    int32_t n_seq, int32_t vocab, float temperature, int32_t* tokens_out,
                                    int64_t* seq_out, void* stream) {
  using namespace ss;
  if (n_seq < 0 || vocab < 1 || !(temperature > 0.f)) return SS_ERR_INVALID_ARG;
  if (vocab > sample::kChunk * sample::kMaxChunks) return SS_ERR_UNSUPPORTED;
  if (n_seq == 0) return SS_OK;
  if (!logits || !draw_offsets || !uniforms || !tokens_out || !seq_out) return SS_ERR_INVALID_ARG;
  SS_LAUNCH(sample::branch_sample_kernel, n_seq, sample::kThreads, 0, as_stream(stream), logits, draw_offsets, uniforms,
            vocab, 1.0 / static_cast<double>(temperature), tokens_out, seq_out);
  return SS_OK;
}
