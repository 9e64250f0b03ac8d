// ss_branch_sample: the sampling half of on-demand branching (paper, Section "Computation Deduplication"): a
// sequence with potential size n draws n next tokens as independent trials from ONE logits row; equal draws are
// grouped afterwards with ss_dedup_paths on (sequence, token) pairs.
//
// One block per sequence, three passes over its logits row (the row stays in L2 after the first):
//   1. maximum                                   (fp32, exact)
//   2. Z = sum_v exp((logit_v - max) / T)        (fp64)
//   3. running CDF in chunks of 4096 tokens (fp64, block scan); every draw whose target u * Z falls into the chunk
//      finds its token with a binary search over the chunk's CDF values in shared memory.
// The decision "first token whose CDF exceeds u * Z" is taken in fp64 so that it agrees with a plain fp64 CPU
// evaluation except for draws within ~1e-15 of a boundary.  Not on the attention hot path: bandwidth is not the aim.
#include "common.cuh"

namespace ss {
namespace sample {

constexpr int kThreads = 1024;
constexpr int kPerThread = 4;
constexpr int kChunk = kThreads * kPerThread;

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
  __shared__ double s_total, s_carry;
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

  // ---- 2. normaliser ------------------------------------------------------------------------------------------------
  double z = 0.0;
  for (int v = tid; v < vocab; v += kThreads) z += exp((static_cast<double>(row[v]) - dmax) * inv_temperature);
  z = warp_sum_d(z);
  if (lane == 0) s_warp[warp] = z;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 32; ++w) t += s_warp[w];
    s_total = t;
  }
  __syncthreads();
  const double Z = s_total;

  // ---- 3. CDF scan; draws are handled in batches of one per thread ------------------------------------------------------
  for (int64_t db = d0; db < d1; db += kThreads) {
    const int64_t d = db + tid;
    const bool have = d < d1;
    const double target = have ? static_cast<double>(uniforms[d]) * Z : 0.0;
    int token = vocab - 1;                                   // the answer if rounding leaves the target above the total
    bool found = !have;
    if (tid == 0) s_carry = 0.0;
    __syncthreads();
    for (int base = 0; base < vocab; base += kChunk) {
      // inclusive CDF of this chunk: thread t owns tokens base + 4t .. base + 4t + 3
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
      const double carry = s_carry;
      double c = carry + (warp ? s_warp[warp - 1] : 0.0) + incl - run;
#pragma unroll
      for (int x = 0; x < kPerThread; ++x) {
        c += e[x];
        s_cdf[tid * kPerThread + x] = c;
      }
      __syncthreads();
      const int n_here = min(kChunk, vocab - base);
      const double chunk_end = s_cdf[n_here - 1];
      if (!found && chunk_end > target) {                    // first index of the chunk whose CDF exceeds the target
        int lo = 0, hi = n_here - 1;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (s_cdf[mid] > target) hi = mid; else lo = mid + 1;
        }
        token = base + lo;
        found = true;
      }
      __syncthreads();
      if (tid == 0) s_carry = chunk_end;
      __syncthreads();
    }
    if (have) {
      tokens_out[d] = token;
      seq_out[d] = s;
    }
  }
}

}  // namespace sample
}  // namespace ss

extern "C" int32_t ss_branch_sample(const float* logits, const int64_t* draw_offsets, const float* uniforms,
                                    int32_t n_seq, int32_t vocab, float temperature, int32_t* tokens_out,
                                    int64_t* seq_out, void* stream) {
  using namespace ss;
  if (n_seq < 0 || vocab < 1 || !(temperature > 0.f)) return SS_ERR_INVALID_ARG;
  if (n_seq == 0) return SS_OK;
  if (!logits || !draw_offsets || !uniforms || !tokens_out || !seq_out) return SS_ERR_INVALID_ARG;
  SS_LAUNCH(sample::branch_sample_kernel, n_seq, sample::kThreads, 0, as_stream(stream), logits, draw_offsets, uniforms,
            vocab, 1.0 / static_cast<double>(temperature), tokens_out, seq_out);
  return SS_OK;
}
