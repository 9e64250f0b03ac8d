// ss_dedup_paths: computation deduplication of candidate paths (paper, Section "Computation Deduplication").
//
// Pipeline (all on the caller's stream, no host synchronisation):
//   1. hash      one warp per path: 64-bit hash of (ctx_key, length, token ids); lanes stride over the tokens,
//                each token is mixed with its position, lane sums are combined with shuffles
//   2. sort      LSD radix sort (8-bit digits, 4 passes) of (top 32 hash bits, path index); stable, so equal
//                keys stay in ascending index order
//   3. match     one warp per sorted position: binary-search the start of its equal-key run, then look for the
//                first earlier run member whose full 64-bit hash, ctx_key, length AND token ids are equal
//                (token ids compared cooperatively by the warp) -> canon
//   4. compact   exclusive scan of (canon[i] == i) in index order -> ranks; unique list, multiplicities
//                (integer atomics: order-independent), path_to_unique, slot remap
// Hash collisions only cost time: equality is always decided on the token ids themselves.
// Batches of up to 4096 paths run the same four steps in two launches (the last block to finish a grid-parallel
// step runs the single-block step that follows it; the sort is a bitonic network in shared memory).
#include "common.cuh"

namespace ss {
namespace dedup {

constexpr int kSortThreads = 256;
constexpr int kSortItems = 8;                       // rounds per tile
constexpr int kSortTile = kSortThreads * kSortItems;
constexpr int kWarpsPerSortBlock = kSortThreads / 32;

__device__ __forceinline__ uint64_t mix64(uint64_t x) {   // splitmix64 finaliser
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
  x ^= x >> 27; x *= 0x94d049bb133111ebull;
  x ^= x >> 31;
  return x;
}

// Whole warp: 64-bit hash of path `path` (returned to every lane).
__device__ __forceinline__ uint64_t hash_path(const int32_t* __restrict__ tok_ids, const int64_t* __restrict__ tok_offsets,
                                              const int64_t* __restrict__ ctx_key, int path, uint32_t weak, int lane) {
  const int64_t lo = tok_offsets[path], hi = tok_offsets[path + 1];
  uint64_t acc = 0;
  for (int64_t j = lo + lane; j < hi; j += 32) {
    const uint64_t t = static_cast<uint32_t>(tok_ids[j]);
    acc += mix64(t * 0x9e3779b97f4a7c15ull + static_cast<uint64_t>(j - lo + 1) * 0xd1b54a32d192ed03ull);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  uint64_t h = mix64(acc ^ mix64(static_cast<uint64_t>(hi - lo) + 0x632be59bd9b4e019ull));
  if (ctx_key) h = mix64(h ^ mix64(static_cast<uint64_t>(ctx_key[path]) + 0x2545f4914f6cdd1dull));
  if (weak) h &= 0xffull;                       // SS_FLAG_WEAK_HASH: force collisions
  return h;
}

__device__ __forceinline__ uint32_t sort_key_of(uint64_t h, uint32_t weak) {
  return weak ? static_cast<uint32_t>(h) : static_cast<uint32_t>(h >> 32);
}

__global__ void hash_kernel(const int32_t* __restrict__ tok_ids, const int64_t* __restrict__ tok_offsets,
                            const int64_t* __restrict__ ctx_key, int n, uint32_t weak, uint64_t* __restrict__ hash64,
                            uint32_t* __restrict__ keys, uint32_t* __restrict__ idx) {
  ss::grid_dependency_enter();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= n) return;
  const uint64_t h = hash_path(tok_ids, tok_offsets, ctx_key, warp, weak, lane);
  if (lane == 0) {
    hash64[warp] = h;
    keys[warp] = sort_key_of(h, weak);
    idx[warp] = warp;
  }
}

// ---- radix sort pass -------------------------------------------------------------------------------------
__global__ void rs_hist(const uint32_t* __restrict__ keys, int n, int shift, int num_tiles, uint32_t* __restrict__ hist) {
  ss::grid_dependency_enter();
  __shared__ uint32_t cnt[256];
  cnt[threadIdx.x] = 0;
  __syncthreads();
  const int base = blockIdx.x * kSortTile;
  for (int r = 0; r < kSortItems; ++r) {
    const int i = base + r * kSortThreads + threadIdx.x;
    if (i < n) atomicAdd(&cnt[(keys[i] >> shift) & 255u], 1u);
  }
  __syncthreads();
  hist[threadIdx.x * num_tiles + blockIdx.x] = cnt[threadIdx.x];
}

// In-place exclusive sum scan of `count` uint32 by one block (looping with a carry).
__global__ void scan_u32_single_block(uint32_t* __restrict__ data, int count) {
  ss::grid_dependency_enter();
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < count; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const uint32_t v = i < count ? data[i] : 0u;
    uint32_t x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) warp_tot[warp] = x;
    __syncthreads();
    if (warp == 0) {
      uint32_t t = lane < nw ? warp_tot[lane] : 0u;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      warp_tot[lane] = t;                         // inclusive totals of warps
    }
    __syncthreads();
    const uint32_t carry = carry_s;
    const uint32_t before = carry + (warp ? warp_tot[warp - 1] : 0u) + x - v;
    if (i < count) data[i] = before;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = before + v;
    __syncthreads();
  }
}

__global__ void rs_scatter(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ idx_in,
                           uint32_t* __restrict__ keys_out, uint32_t* __restrict__ idx_out, int n, int shift,
                           int num_tiles, const uint32_t* __restrict__ hist) {
  ss::grid_dependency_enter();
  __shared__ uint32_t base[256];
  __shared__ uint32_t wc[kWarpsPerSortBlock][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  base[threadIdx.x] = hist[threadIdx.x * num_tiles + blockIdx.x];
#pragma unroll
  for (int w = 0; w < kWarpsPerSortBlock; ++w) wc[w][threadIdx.x] = 0;
  __syncthreads();
  const int tile_base = blockIdx.x * kSortTile;
  for (int r = 0; r < kSortItems; ++r) {
    const int i = tile_base + r * kSortThreads + threadIdx.x;
    const bool valid = i < n;
    uint32_t key = 0, id = 0;
    if (valid) { key = keys_in[i]; id = idx_in[i]; }
    const uint32_t digit = valid ? ((key >> shift) & 255u) : 256u;
    const uint32_t peers = __match_any_sync(0xffffffffu, digit);
    const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
    if (valid && rank == 0) wc[warp][digit] = __popc(peers);
    __syncthreads();
    if (valid) {
      uint32_t off = base[digit] + rank;
      for (int w = 0; w < warp; ++w) off += wc[w][digit];
      keys_out[off] = key;
      idx_out[off] = id;
    }
    __syncthreads();
    {
      uint32_t tot = 0;
#pragma unroll
      for (int w = 0; w < kWarpsPerSortBlock; ++w) { tot += wc[w][threadIdx.x]; wc[w][threadIdx.x] = 0; }
      base[threadIdx.x] += tot;
    }
    __syncthreads();
  }
}

// ---- exact matching inside equal-key runs ---------------------------------------------------------------
// Whole warp: canonical representative of the path at sorted position s.
// (keys, idx, hash64 carry no __restrict__ here: the single-block kernel writes them before it reads them.)
__device__ __forceinline__ void match_sorted_position(const uint32_t* keys, const uint32_t* idx, int s,
                                                      const uint64_t* hash64,
                                                      const int32_t* __restrict__ tok_ids,
                                                      const int64_t* __restrict__ tok_offsets,
                                                      const int64_t* __restrict__ ctx_key,
                                                      int32_t* canon_out, int lane) {
  const uint32_t key = keys[s];
  const int i = static_cast<int>(idx[s]);
  // start of the run of equal keys (lower bound)
  int lo = 0, hi = s;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (keys[mid] < key) lo = mid + 1; else hi = mid;
  }
  const uint64_t hi_ = hash64[i];
  const int64_t a0 = tok_offsets[i], alen = tok_offsets[i + 1] - a0;
  const int64_t actx = ctx_key ? ctx_key[i] : 0;
  int canon = i;
  for (int b = lo; b < s && canon == i; b += 32) {
    const int t = b + lane;
    bool cand = false;
    int j = 0;
    if (t < s) {
      j = static_cast<int>(idx[t]);
      cand = hash64[j] == hi_ && (tok_offsets[j + 1] - tok_offsets[j]) == alen && (ctx_key ? ctx_key[j] : 0) == actx;
    }
    uint32_t m = __ballot_sync(0xffffffffu, cand);
    while (m) {
      const int src = __ffs(m) - 1;
      m &= m - 1;
      const int jj = __shfl_sync(0xffffffffu, j, src);
      const int64_t b0 = tok_offsets[jj];
      bool same = true;
      for (int64_t p = 0; p < alen && same; p += 32) {
        const int64_t q = p + lane;
        const bool eq = q < alen ? (tok_ids[a0 + q] == tok_ids[b0 + q]) : true;
        same = __all_sync(0xffffffffu, eq);
      }
      if (same) { canon = jj; break; }
    }
  }
  if (lane == 0) canon_out[i] = canon;
}

__global__ void match_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ idx, int n,
                             const uint64_t* __restrict__ hash64, const int32_t* __restrict__ tok_ids,
                             const int64_t* __restrict__ tok_offsets, const int64_t* __restrict__ ctx_key,
                             int32_t* __restrict__ canon_out) {
  ss::grid_dependency_enter();
  const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (s >= n) return;
  match_sorted_position(keys, idx, s, hash64, tok_ids, tok_offsets, ctx_key, canon_out, threadIdx.x & 31);
}

// ---- compaction ----------------------------------------------------------------------------------------------
// One block: rank[i] = number of unique paths with a smaller index; also clears the multiplicities.
__device__ __forceinline__ void rank_block(const int32_t* canon, int n, int32_t* rank, int32_t* multiplicity,
                                           int32_t* num_unique) {
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = (i < n && canon[i] == i) ? 1 : 0;
    if (i < n) multiplicity[i] = 0;
    const uint32_t bal = __ballot_sync(0xffffffffu, v);
    const int incl_w = __popc(bal & (0xffffffffu >> (31 - lane)));
    if (lane == 31) warp_tot[warp] = incl_w;
    __syncthreads();
    if (warp == 0) {
      int t = lane < nw ? warp_tot[lane] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      warp_tot[lane] = t;
    }
    __syncthreads();
    const int before = carry_s + (warp ? warp_tot[warp - 1] : 0) + incl_w - v;
    if (i < n) rank[i] = before;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) *num_unique = carry_s;
}

__global__ void rank_kernel(const int32_t* __restrict__ canon, int n, int32_t* __restrict__ rank,
                            int32_t* __restrict__ multiplicity, int32_t* __restrict__ num_unique) {
  ss::grid_dependency_enter();
  rank_block(canon, n, rank, multiplicity, num_unique);
}

__device__ __forceinline__ void finalize_path(const int32_t* canon, const int32_t* rank, int i,
                                              const int32_t* __restrict__ slot_in, int32_t* path_to_unique,
                                              int32_t* unique_paths, int32_t* multiplicity, int32_t* slot_out) {
  const int c = canon[i];
  const int r = rank[c];
  path_to_unique[i] = r;
  if (c == i) unique_paths[r] = i;
  atomicAdd(&multiplicity[r], 1);
  if (slot_out) slot_out[i] = slot_in[c];
}

__global__ void finalize_kernel(const int32_t* __restrict__ canon, const int32_t* __restrict__ rank, int n,
                                const int32_t* __restrict__ slot_in, int32_t* __restrict__ path_to_unique,
                                int32_t* __restrict__ unique_paths, int32_t* __restrict__ multiplicity,
                                int32_t* __restrict__ slot_out) {
  ss::grid_dependency_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  finalize_path(canon, rank, i, slot_in, path_to_unique, unique_paths, multiplicity, slot_out);
}

// ---- small batches ---------------------------------------------------------------------------------------------
// A batch of a few thousand paths is launch-latency bound: the multi-launch path above is ~17 dependent launches.
// Here the same four steps take two: the grid-parallel steps (hash, match) stay grid-parallel, and the block that
// finishes LAST (a counter in the workspace, zeroed by a memset ahead of the first kernel) runs the single-block step
// that follows (bitonic sort in shared memory; rank scan + finalize).
constexpr int kSmallMax = 4096;
constexpr int kSmallThreads = 1024;
constexpr int kSmallWarps = kSmallThreads / 32;

// True in every thread of the block that arrives last; its reads come after all other blocks' writes.
__device__ __forceinline__ bool last_block_arrives(unsigned int* counter) {
  __shared__ bool s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(counter, 1u) == gridDim.x - 1;
  __syncthreads();
  if (s_last) __threadfence();
  return s_last;
}

// Sort by counting, for batches too large for one block's shared-memory sort and too small to be worth a radix sort's
// twelve launches: the rank of a path is the number of paths with a smaller (sort key, index) pair, counted by brute
// force - n^2 comparisons, 0.27 G at 16384 paths, spread over the whole device (a few microseconds), against a
// bitonic sort by a single block (~0.25 ms there: one SM, a hundred barrier-separated stages).  One thread per path;
// the keys go through shared memory in tiles.
constexpr int kRankThreads = 256;
constexpr int kRankTile = 2048;
constexpr int kRankSortMax = 32768;

// Block (bi, bj) counts, for the 256 paths of group bi, the smaller pairs among the 2048 paths of tile bj and adds
// the counts to rank_acc[] (zeroed before the launch); the block that completes a group - the last of its tiles to
// arrive at group_done[bi] - scatters the group's keys and indices to their ranks.
__global__ void __launch_bounds__(kRankThreads)
rank_sort_kernel(const uint32_t* __restrict__ keys_in, int n, int n_tiles, int* rank_acc, unsigned int* group_done,
                 uint32_t* __restrict__ keys_out, uint32_t* __restrict__ idx_out) {
  ss::grid_dependency_enter();
  __shared__ __align__(16) uint32_t tile[kRankTile];
  __shared__ bool s_last;
  const int bi = blockIdx.x / n_tiles, bj = blockIdx.x - bi * n_tiles;
  const int i = bi * kRankThreads + threadIdx.x;
  const uint32_t k = i < n ? keys_in[i] : 0xffffffffu;
  const int base = bj * kRankTile;
  for (int t = threadIdx.x; t < kRankTile; t += kRankThreads) tile[t] = base + t < n ? keys_in[base + t] : 0xffffffffu;
  __syncthreads();
  int cnt = 0;
  // paths before this one count when their key is <= k, paths after it when it is < k (ties go by index); a tile
  // that lies wholly on one side of the group's own paths takes the cheap uniform loop
  if (base + kRankTile <= bi * kRankThreads) {
#pragma unroll 4
    for (int t = 0; t < kRankTile; t += 4) {
      const uint4 v = *reinterpret_cast<const uint4*>(&tile[t]);
      cnt += (v.x <= k) + (v.y <= k) + (v.z <= k) + (v.w <= k);
    }
  } else if (base >= (bi + 1) * kRankThreads) {
#pragma unroll 4
    for (int t = 0; t < kRankTile; t += 4) {         // (padding entries are 0xffffffff: never < k)
      const uint4 v = *reinterpret_cast<const uint4*>(&tile[t]);
      cnt += (v.x < k) + (v.y < k) + (v.z < k) + (v.w < k);
    }
  } else {
    const int n_here = min(kRankTile, n - base);
    for (int t = 0; t < n_here; ++t) cnt += (tile[t] < k) || (tile[t] == k && base + t < i);
  }
  if (i < n && cnt) atomicAdd(&rank_acc[i], cnt);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&group_done[bi], 1u) == static_cast<unsigned>(n_tiles - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (i < n) {
    const int rank = __ldcg(&rank_acc[i]);
    keys_out[rank] = k;
    idx_out[rank] = static_cast<uint32_t>(i);
  }
}

__global__ void __launch_bounds__(kSmallThreads)
small_hash_sort_kernel(const int32_t* __restrict__ tok_ids, const int64_t* __restrict__ tok_offsets,
                       const int64_t* __restrict__ ctx_key, int n, uint32_t weak, uint64_t* hash64, uint32_t* keys,
                       uint32_t* idx, unsigned int* counter) {
  ss::grid_dependency_enter();
  __shared__ uint64_t skey[kSmallMax];            // (sort key << 32 | path index): distinct, so the order is total
  const int tid = threadIdx.x, lane = tid & 31;
  const int p = blockIdx.x * kSmallWarps + (tid >> 5);
  if (p < n) {
    const uint64_t h = hash_path(tok_ids, tok_offsets, ctx_key, p, weak, lane);
    if (lane == 0) hash64[p] = h;
  }
  if (!last_block_arrives(counter)) return;
  int n_pad = 1;
  while (n_pad < n) n_pad <<= 1;
  for (int i = tid; i < n_pad; i += blockDim.x)
    skey[i] = i < n ? (static_cast<uint64_t>(sort_key_of(__ldcg(hash64 + i), weak)) << 32) | static_cast<uint32_t>(i)
                    : ~0ull;
  __syncthreads();
  for (int size = 2; size <= n_pad; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int t = tid; t < (n_pad >> 1); t += blockDim.x) {
        const int lo = ((t / stride) * (stride << 1)) + (t % stride);
        const int hi = lo + stride;
        const bool up = ((lo & size) == 0);
        const uint64_t a = skey[lo], b = skey[hi];
        if ((a > b) == up) { skey[lo] = b; skey[hi] = a; }
      }
      __syncthreads();
    }
  for (int i = tid; i < n; i += blockDim.x) {
    keys[i] = static_cast<uint32_t>(skey[i] >> 32);
    idx[i] = static_cast<uint32_t>(skey[i]);
  }
}

__global__ void __launch_bounds__(kSmallThreads)
small_match_finalize_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ idx, int n,
                            const uint64_t* __restrict__ hash64, const int32_t* __restrict__ tok_ids,
                            const int64_t* __restrict__ tok_offsets, const int64_t* __restrict__ ctx_key,
                            const int32_t* __restrict__ slot_in, int32_t* canon_out, int32_t* rank,
                            int32_t* path_to_unique, int32_t* unique_paths, int32_t* multiplicity, int32_t* slot_out,
                            int32_t* num_unique, unsigned int* counter) {
  ss::grid_dependency_enter();
  const int s = blockIdx.x * kSmallWarps + (threadIdx.x >> 5);
  if (s < n) match_sorted_position(keys, idx, s, hash64, tok_ids, tok_offsets, ctx_key, canon_out, threadIdx.x & 31);
  if (!last_block_arrives(counter)) return;
  rank_block(canon_out, n, rank, multiplicity, num_unique);     // canon_out was not read before: no stale L1 lines
  __syncthreads();
  for (int i = threadIdx.x; i < n; i += blockDim.x)
    finalize_path(canon_out, rank, i, slot_in, path_to_unique, unique_paths, multiplicity, slot_out);
}

// ---- ss_gather_unique_paths ------------------------------------------------------------------------------------
// One block.  Thread t owns kGatherItems consecutive unique paths per round: it gathers their descriptor rows and the
// block scans the query lengths (thread sums -> warp shuffles -> warp totals -> running carry).
constexpr int kGatherThreads = 1024;
constexpr int kGatherItems = 4;       // (16 per thread - one round for 16384 paths - was measured: 33 -> 60 us, every access 32 sectors wide)

__global__ void __launch_bounds__(kGatherThreads)
gather_unique_kernel(const int32_t* __restrict__ unique_paths, const int32_t* __restrict__ num_unique, int n,
                     const int32_t* __restrict__ path_leaf_node, const int32_t* __restrict__ path_q_len,
                     const int64_t* __restrict__ q_offsets, int32_t* __restrict__ u_leaf, int32_t* __restrict__ u_q_len,
                     int64_t* __restrict__ u_q_offsets, int64_t* __restrict__ u_q_src) {
  ss::grid_dependency_enter();
  __shared__ long long warp_tot[32];
  __shared__ long long carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int U = min(max(*num_unique, 0), n);
  if (threadIdx.x == 0) { carry_s = 0; u_q_offsets[0] = 0; }
  __syncthreads();
  for (int base = 0; base < n; base += kGatherThreads * kGatherItems) {
    const int p0 = base + threadIdx.x * kGatherItems;
    int len[kGatherItems];
    long long mine = 0;
#pragma unroll
    for (int e = 0; e < kGatherItems; ++e) {
      const int p = p0 + e;
      len[e] = 0;
      if (p < n) {
        int leaf = -1;
        long long src_row = 0;
        if (p < U) {
          const int src = unique_paths[p];
          leaf = path_leaf_node[src];
          len[e] = path_q_len[src];
          src_row = q_offsets[src];
        }
        u_leaf[p] = leaf;
        u_q_len[p] = len[e];
        u_q_src[p] = src_row;
      }
      mine += len[e];
    }
    long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      long long t = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      warp_tot[lane] = t;
    }
    __syncthreads();
    long long run = carry_s + (warp ? warp_tot[warp - 1] : 0) + incl - mine;   // rows before path p0
#pragma unroll
    for (int e = 0; e < kGatherItems; ++e) {
      run += len[e];
      if (p0 + e < n) u_q_offsets[p0 + e + 1] = run;
    }
    __syncthreads();
    if (threadIdx.x == kGatherThreads - 1) carry_s = run;
    __syncthreads();
  }
}

__global__ void zero_scalar_kernel(int32_t* p) {
  ss::grid_dependency_enter(); *p = 0; }

struct Layout {
  size_t hash64, keys_a, keys_b, idx_a, idx_b, hist, rank, total;
  int num_tiles;
};

static Layout layout(int n) {
  Layout L;
  const size_t m = n > 0 ? n : 1;
  L.num_tiles = static_cast<int>((m + kSortTile - 1) / kSortTile);
  size_t off = 0;
  L.hash64 = off; off = align_up(off + m * 8);
  L.keys_a = off; off = align_up(off + m * 4);
  L.keys_b = off; off = align_up(off + m * 4);
  L.idx_a = off; off = align_up(off + m * 4);
  L.idx_b = off; off = align_up(off + m * 4);
  L.hist = off; off = align_up(off + static_cast<size_t>(256) * L.num_tiles * 4);
  L.rank = off; off = align_up(off + m * 4);
  L.total = off;
  return L;
}

}  // namespace dedup
}  // namespace ss

extern "C" int32_t ss_dedup_workspace_bytes(int32_t n_paths, size_t* out_bytes) {
  if (n_paths < 0 || !out_bytes) return SS_ERR_INVALID_ARG;
  *out_bytes = ss::dedup::layout(n_paths).total;
  return SS_OK;
}

extern "C" int32_t ss_dedup_paths(const int32_t* tok_ids, const int64_t* tok_offsets, const int64_t* ctx_key,
                                  const int32_t* slot_in, int32_t n_paths, uint32_t flags, int32_t* canon_out,
                                  int32_t* path_to_unique_out, int32_t* unique_paths_out,
                                  int32_t* multiplicity_out, int32_t* slot_out, int32_t* num_unique_out,
                                  void* workspace, size_t workspace_bytes, void* stream) {
  using namespace ss;
  using namespace ss::dedup;
  if (n_paths < 0 || !num_unique_out) return SS_ERR_INVALID_ARG;
  if (flags & ~SS_FLAG_WEAK_HASH) return SS_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (n_paths == 0) {
    SS_LAUNCH(zero_scalar_kernel, 1, 1, 0, st, num_unique_out);
    return SS_OK;
  }
  if ((slot_in == nullptr) != (slot_out == nullptr)) return SS_ERR_INVALID_ARG;
  if (!tok_offsets || !canon_out || !path_to_unique_out || !unique_paths_out || !multiplicity_out || !workspace)
    return SS_ERR_INVALID_ARG;
  if (!tok_ids) return SS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return SS_ERR_INVALID_ARG;
  const Layout L = layout(n_paths);
  if (workspace_bytes < L.total) return SS_ERR_WORKSPACE_TOO_SMALL;
  char* ws = static_cast<char*>(workspace);
  uint64_t* hash64 = reinterpret_cast<uint64_t*>(ws + L.hash64);
  uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + L.keys_a);
  uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + L.keys_b);
  uint32_t* idx_a = reinterpret_cast<uint32_t*>(ws + L.idx_a);
  uint32_t* idx_b = reinterpret_cast<uint32_t*>(ws + L.idx_b);
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + L.hist);
  int32_t* rank = reinterpret_cast<int32_t*>(ws + L.rank);

  const int n = n_paths;
  const uint32_t weak = (flags & SS_FLAG_WEAK_HASH) ? 1u : 0u;
  if (n <= kSmallMax) {
    unsigned int* counters = reinterpret_cast<unsigned int*>(hist);      // the sort histogram is unused on this path
    if (cudaMemsetAsync(counters, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    const int blocks = (n + kSmallWarps - 1) / kSmallWarps;
    SS_LAUNCH(small_hash_sort_kernel, blocks, kSmallThreads, 0, st, tok_ids, tok_offsets, ctx_key, n, weak, hash64, keys_a,
              idx_a, counters);
    SS_LAUNCH(small_match_finalize_kernel, blocks, kSmallThreads, 0, st, keys_a, idx_a, n, hash64, tok_ids, tok_offsets,
              ctx_key, slot_in, canon_out, rank, path_to_unique_out, unique_paths_out, multiplicity_out, slot_out,
              num_unique_out, counters + 1);
    return SS_OK;
  }
  const int warps_per_block = 8;
  const int warp_blocks = (n + warps_per_block - 1) / warps_per_block;
  SS_LAUNCH(hash_kernel, warp_blocks, warps_per_block * 32, 0, st, tok_ids, tok_offsets, ctx_key, n, weak, hash64,
            keys_a, idx_a);
  if (n <= kRankSortMax) {                          // three launches: hash, sort by counting, match + rank + finalize
    unsigned int* counters = reinterpret_cast<unsigned int*>(hist);      // the sort histogram is unused on this path
    if (cudaMemsetAsync(counters, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    // (idx_a holds the identity permutation the radix sort starts from: free here, it accumulates the ranks; the
    //  group counters follow the two arrival counters in the histogram region)
    const int n_groups = (n + kRankThreads - 1) / kRankThreads, n_tiles = (n + kRankTile - 1) / kRankTile;
    if (cudaMemsetAsync(idx_a, 0, static_cast<size_t>(n) * sizeof(uint32_t), st) != cudaSuccess ||
        cudaMemsetAsync(counters + 2, 0, static_cast<size_t>(n_groups) * sizeof(unsigned int), st) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    SS_LAUNCH(rank_sort_kernel, n_groups * n_tiles, kRankThreads, 0, st, keys_a, n, n_tiles, reinterpret_cast<int*>(idx_a),
              counters + 2, keys_b, idx_b);
    SS_LAUNCH(small_match_finalize_kernel, (n + kSmallWarps - 1) / kSmallWarps, kSmallThreads, 0, st, keys_b, idx_b, n,
              hash64, tok_ids, tok_offsets, ctx_key, slot_in, canon_out, rank, path_to_unique_out, unique_paths_out,
              multiplicity_out, slot_out, num_unique_out, counters + 1);
    return SS_OK;
  }
  const int passes = weak ? 1 : 4;
  uint32_t *kin = keys_a, *kout = keys_b, *iin = idx_a, *iout = idx_b;
  for (int p = 0; p < passes; ++p) {
    const int shift = 8 * p;
    SS_LAUNCH(rs_hist, L.num_tiles, kSortThreads, 0, st, kin, n, shift, L.num_tiles, hist);
    SS_LAUNCH(scan_u32_single_block, 1, 1024, 0, st, hist, 256 * L.num_tiles);
    SS_LAUNCH(rs_scatter, L.num_tiles, kSortThreads, 0, st, kin, iin, kout, iout, n, shift, L.num_tiles, hist);
    uint32_t* t = kin; kin = kout; kout = t;
    t = iin; iin = iout; iout = t;
  }
  SS_LAUNCH(match_kernel, warp_blocks, warps_per_block * 32, 0, st, kin, iin, n, hash64, tok_ids, tok_offsets,
            ctx_key, canon_out);
  SS_LAUNCH(rank_kernel, 1, 1024, 0, st, canon_out, n, rank, multiplicity_out, num_unique_out);
  SS_LAUNCH(finalize_kernel, (n + 255) / 256, 256, 0, st, canon_out, rank, n, slot_in, path_to_unique_out,
            unique_paths_out, multiplicity_out, slot_out);
  return SS_OK;
}

// ---------------------------------------------------------------------------------------------------------
// ss_dedup_paths_static: the same deduplication for callers that must not allocate device memory.
//
// Some hosts of this library cannot obtain scratch memory at the moment they need a deduplication pass: a serving
// engine that has already handed all free HBM to its KV-cache pool (an allocation would fail, or shrink the cache),
// a latency-critical scheduling loop in which the device-wide synchronisation hidden in an allocation is not
// acceptable, or a plug-in that is simply not allowed to touch the allocator.  For them the scratch lives in the
// library image itself: a fixed array in device global memory, present on every GPU that loads the library, from
// load until the process ends.
//
// In host code the array's name below is only a handle for the runtime, not a device address; the address that
// kernels can use is obtained once per device with cudaGetSymbolAddress (with that device current) and cached.
// ---------------------------------------------------------------------------------------------------------
namespace ss {
namespace dedup {

constexpr int kStaticMaxPaths = SS_DEDUP_STATIC_MAX_PATHS;
constexpr size_t kStaticScratchBytes = 2u << 20;           // 2 MiB; layout(kStaticMaxPaths).total is about 1.8 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_static_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (looked up on the first call per device).
static int32_t static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return SS_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return SS_ERR_UNSUPPORTED;
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = ptr;
  }
  *out = g_static_scratch_addr[dev];
  return SS_OK;
}

}  // namespace dedup
}  // namespace ss

extern "C" int32_t ss_dedup_paths_static(const int32_t* tok_ids, const int64_t* tok_offsets, const int64_t* ctx_key,
                                         const int32_t* slot_in, int32_t n_paths, uint32_t flags, int32_t* canon_out,
                                         int32_t* path_to_unique_out, int32_t* unique_paths_out,
                                         int32_t* multiplicity_out, int32_t* slot_out, int32_t* num_unique_out,
                                         void* stream) {
  using namespace ss::dedup;
  if (n_paths < 0) return SS_ERR_INVALID_ARG;
  if (n_paths > kStaticMaxPaths) return SS_ERR_UNSUPPORTED;          // larger batches need ss_dedup_paths
  if (layout(n_paths).total > kStaticScratchBytes) return SS_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  const int32_t rc = static_scratch_address(&scratch);
  if (rc != SS_OK) return rc;
  // Nothing in the scratch has to start at zero: every region is fully written before it is read (histograms,
  // keys, ranks), and the multiplicities that do start at zero are an output cleared by the rank kernel.
  return ss_dedup_paths(tok_ids, tok_offsets, ctx_key, slot_in, n_paths, flags, canon_out, path_to_unique_out,
                        unique_paths_out, multiplicity_out, slot_out, num_unique_out, scratch, kStaticScratchBytes,
                        stream);
}

extern "C" int32_t ss_gather_unique_paths(const int32_t* unique_paths, const int32_t* num_unique, int32_t n_paths,
                                          const int32_t* path_leaf_node, const int32_t* path_q_len,
                                          const int64_t* q_offsets, int32_t* u_leaf_out, int32_t* u_q_len_out,
                                          int64_t* u_q_offsets_out, int64_t* u_q_src_out, void* stream) {
  using namespace ss;
  using namespace ss::dedup;
  if (n_paths < 0 || !u_q_offsets_out) return SS_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  if (n_paths == 0) {
    if (cudaMemsetAsync(u_q_offsets_out, 0, sizeof(int64_t), st) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    return SS_OK;
  }
  if (!unique_paths || !num_unique || !path_leaf_node || !path_q_len || !q_offsets || !u_leaf_out || !u_q_len_out ||
      !u_q_src_out)
    return SS_ERR_INVALID_ARG;
  SS_LAUNCH(gather_unique_kernel, 1, kGatherThreads, 0, st, unique_paths, num_unique, n_paths, path_leaf_node, path_q_len,
            q_offsets, u_leaf_out, u_q_len_out, u_q_offsets_out, u_q_src_out);
  return SS_OK;
}
