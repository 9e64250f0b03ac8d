// ss_build_prefix_tree: radix tree of candidate paths over whole KV pages, from raw token ids (paper, Section
// "Computation Deduplication": candidates of a step share a large part of their tokens; Section "Experimental Setup":
// prefix KV caching and sharing).  Only whole pages are shared; every path gets a private leaf node.
//
// Pipeline (all on the caller's stream, no host synchronisation):
//   1. page hashes   one warp per path: 64-bit hash of every full page (lanes take pages, 64 contiguous bytes each),
//                    chained into prefix hashes H[k] = hash of the first k pages
//   2. sort          bitonic sort of the path indices by token sequence.  The comparator finds the number of common
//                    pages of two paths by binary search over their prefix hashes and then compares tokens from there,
//                    so a comparison costs O(log pages) whatever the length of the common prefix.  Blocks of 2048
//                    indices are sorted in shared memory; larger strides take one launch each.
//   3. neighbours    one warp per sorted neighbour pair: the common full pages are counted on the TOKENS themselves
//                    (the hashes only ordered the paths), and the order of the pair is checked; a hash collision that
//                    mis-ordered two paths is reported as SS_ERR_BAD_INPUT instead of producing a wrong tree
//   4. tree          inner nodes are the intervals of neighbours that share more pages than their surroundings (the
//                    LCP-interval tree).  One thread per position: it finds its interval with nearest-smaller-value
//                    searches that skip whole blocks through their minima; depth-first numbering (leaves included)
//                    comes from a prefix sum of the intervals per start rank; parents follow from the neighbours of
//                    an interval
#include "common.cuh"

namespace ss {
namespace ptree {

constexpr int kSortBlock = 1024;                 // threads; a block sorts 2048 indices in shared memory
constexpr int kSortChunk = 2 * kSortBlock;

__device__ __forceinline__ uint64_t mix64(uint64_t x) {   // splitmix64 finaliser
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
  x ^= x >> 27; x *= 0x94d049bb133111ebull;
  x ^= x >> 31;
  return x;
}

struct Seqs {
  const int32_t* tok_ids;
  const int64_t* tok_offsets;
  const uint64_t* hashes;       // prefix hashes, path i at hashes[hash_base(i) + k], k = 0 .. full pages of i
  int page;
};

// Prefix hashes of path i start here: (offset / page) + i never overlaps the previous path's (pages + 1) entries.
__device__ __forceinline__ int64_t hash_base(const Seqs& S, int i) {
  return (S.tok_offsets[i] - S.tok_offsets[0]) / S.page + i;
}

// ---- 1. page hashes -----------------------------------------------------------------------------------------------
__global__ void page_hash_kernel(const int32_t* __restrict__ tok_ids, const int64_t* __restrict__ tok_offsets, int n,
                                 int page, uint64_t* __restrict__ hashes) {
  ss::grid_dependency_enter();
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (i >= n) return;
  const int64_t t0 = tok_offsets[i];
  const int n_pages = static_cast<int>((tok_offsets[i + 1] - t0) / page);
  uint64_t* H = hashes + ((t0 - tok_offsets[0]) / page + i);
  uint64_t h = 0x9e3779b97f4a7c15ull;                       // H[0]: the empty prefix
  if (lane == 0) H[0] = h;
  for (int k0 = 0; k0 < n_pages; k0 += 32) {
    const int k = k0 + lane;
    uint64_t c = 0;
    if (k < n_pages) {
      const int32_t* p = tok_ids + t0 + static_cast<int64_t>(k) * page;
      for (int t = 0; t < page; ++t) c = mix64(c ^ (static_cast<uint64_t>(static_cast<uint32_t>(p[t])) + 0x632be59bd9b4e019ull * (t + 1)));
    }
    const int m = min(32, n_pages - k0);
    for (int x = 0; x < m; ++x) {                           // the chain is sequential: every lane follows it
      const uint64_t cx = __shfl_sync(0xffffffffu, c, x);
      h = mix64(h ^ cx);
      if (lane == x) H[k0 + x + 1] = h;
    }
  }
}

// ---- 2. sort --------------------------------------------------------------------------------------------------------
// Strict order of two distinct paths: token sequence, a proper prefix first, then the index.  -1 is the padding
// index and sorts last.
__device__ bool path_less(const Seqs& S, int a, int b) {
  if (a < 0 || b < 0) return b < 0 && a >= 0;
  const int64_t a0 = S.tok_offsets[a], b0 = S.tok_offsets[b];
  const int64_t la = S.tok_offsets[a + 1] - a0, lb = S.tok_offsets[b + 1] - b0;
  const uint64_t* Ha = S.hashes + hash_base(S, a);
  const uint64_t* Hb = S.hashes + hash_base(S, b);
  int lo = 0, hi = static_cast<int>(min(la, lb) / S.page);  // common pages: H equal at lo, (unknown) above
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (Ha[mid] == Hb[mid]) lo = mid; else hi = mid - 1;
  }
  const int64_t n = min(la, lb);
  for (int64_t t = static_cast<int64_t>(lo) * S.page; t < n; ++t) {
    const int32_t x = S.tok_ids[a0 + t], y = S.tok_ids[b0 + t];
    if (x != y) return x < y;
  }
  if (la != lb) return la < lb;
  return a < b;
}

__device__ __forceinline__ void compare_exchange(const Seqs& S, int& x, int& y, bool up) {
  if (path_less(S, y, x) == up) { const int t = x; x = y; y = t; }
}

// Compare-exchange passes at distances first_stride, first_stride / 2, .. 1 inside a chunk held in shared memory;
// `size` is the bitonic merge they belong to (it fixes the direction of every pair).
__device__ __forceinline__ void local_passes(const Seqs& S, int* s, int base, int size, int first_stride) {
  for (int stride = first_stride; stride > 0; stride >>= 1) {
    const int t = threadIdx.x;
    const int lo = ((t / stride) * (stride << 1)) + (t % stride);
    const int hi = lo + stride;
    const bool up = (((base + lo) & size) == 0);
    int x = s[lo], y = s[hi];
    compare_exchange(S, x, y, up);
    s[lo] = x; s[hi] = y;
    __syncthreads();
  }
}

// size == 0: sorts every chunk of kSortChunk indices completely (merges of size 2 .. kSortChunk).
// size  > kSortChunk: the tail of the merge of that size (distances below a chunk), after merge_step_kernel has done
// the distances of a chunk and above.
__global__ void __launch_bounds__(kSortBlock)
sort_chunks_kernel(Seqs S, int* __restrict__ idx, int n_pad, int size) {
  ss::grid_dependency_enter();
  __shared__ int s[kSortChunk];
  const int base = blockIdx.x * kSortChunk;
  for (int t = threadIdx.x; t < kSortChunk; t += kSortBlock) s[t] = base + t < n_pad ? idx[base + t] : -1;
  __syncthreads();
  if (size == 0) {
    for (int sz = 2; sz <= kSortChunk; sz <<= 1) local_passes(S, s, base, sz, sz >> 1);
  } else {
    local_passes(S, s, base, size, kSortChunk >> 1);
  }
  for (int t = threadIdx.x; t < kSortChunk; t += kSortBlock)
    if (base + t < n_pad) idx[base + t] = s[t];
}

// One compare-exchange pass of the merge of size `size` at distance `stride` (>= kSortChunk).
__global__ void merge_step_kernel(Seqs S, int* __restrict__ idx, int n_pad, int size, int stride) {
  ss::grid_dependency_enter();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (n_pad >> 1)) return;
  const int lo = ((t / stride) * (stride << 1)) + (t % stride);
  const int hi = lo + stride;
  const bool up = ((lo & size) == 0);
  int x = idx[lo], y = idx[hi];
  const int x0 = x;
  compare_exchange(S, x, y, up);
  if (x != x0) { idx[lo] = x; idx[hi] = y; }
}

__global__ void iota_kernel(int* __restrict__ idx, int n, int n_pad) {
  ss::grid_dependency_enter();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n_pad) idx[t] = t < n ? t : -1;
}

// ---- 3. neighbours --------------------------------------------------------------------------------------------------
// lcp[r] = full pages shared by the paths of rank r-1 and r (lcp[0] = 0), counted on the tokens; also checks that the
// pair is in order (a hash collision could have mis-ordered it).
__global__ void neighbour_kernel(Seqs S, const int* __restrict__ idx, int n, int* __restrict__ lcp,
                                 int32_t* __restrict__ order_out, int32_t* __restrict__ status) {
  ss::grid_dependency_enter();
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (r >= n) return;
  const int b = idx[r];
  if (lane == 0) order_out[r] = b;
  if (r == 0) {
    if (lane == 0) lcp[0] = 0;
    return;
  }
  const int a = idx[r - 1];
  const int64_t a0 = S.tok_offsets[a], b0 = S.tok_offsets[b];
  const int64_t la = S.tok_offsets[a + 1] - a0, lb = S.tok_offsets[b + 1] - b0;
  const int64_t m = min(la, lb);
  int64_t d = m;                                            // first differing position
  for (int64_t t0 = 0; t0 < m; t0 += 32) {
    const int64_t t = t0 + lane;
    const bool ne = t < m && S.tok_ids[a0 + t] != S.tok_ids[b0 + t];
    const uint32_t bal = __ballot_sync(0xffffffffu, ne);
    if (bal) { d = t0 + __ffs(bal) - 1; break; }
  }
  if (lane == 0) {
    lcp[r] = static_cast<int>(d / S.page);
    bool in_order;
    if (d < m) in_order = S.tok_ids[a0 + d] < S.tok_ids[b0 + d];
    else in_order = la < lb || (la == lb && a < b);
    if (!in_order) set_status(status, SS_ERR_BAD_INPUT);
  }
}

// ---- 4. tree ---------------------------------------------------------------------------------------------------------
// Inner nodes are the LCP intervals of lcp[]: maximal runs of ranks a..b whose neighbours all share at least d pages
// (lcp[a+1..b] >= d, with equality somewhere) while lcp[a] < d and lcp[b+1] < d (lcp[n] counts as 0).  The interval is
// created by its first position x with lcp[x] == d.  Everything below is one thread per position / rank with
// nearest-smaller-value searches over lcp[], which skip whole blocks of kMinBlock entries through their minima.
constexpr int kMinBlock = 256;

struct Lcp {
  const int* v;        // lcp[0..n)
  const int* bmin;     // minimum of every block of kMinBlock entries
  int n;
};

// Largest p < x with lcp[p] < bound (STRICT) or <= bound; lcp[0] = 0 ends every search for bound >= 0 (> 0 if strict).
template <bool STRICT>
__device__ int prev_below(const Lcp& L, int x, int bound) {
  auto hit = [&](int val) { return STRICT ? val < bound : val <= bound; };
  int p = x - 1;
  const int blk_lo = (x / kMinBlock) * kMinBlock;
  for (; p >= blk_lo; --p)
    if (hit(L.v[p])) return p;
  int blk = x / kMinBlock - 1;
  while (blk > 0 && !hit(L.bmin[blk])) --blk;
  for (p = blk * kMinBlock + kMinBlock - 1; p > 0; --p)
    if (hit(L.v[p])) return p;
  return 0;
}
// Smallest q > x with lcp[q] < bound (STRICT) or <= bound; n if there is none.
template <bool STRICT>
__device__ int next_below(const Lcp& L, int x, int bound) {
  auto hit = [&](int val) { return STRICT ? val < bound : val <= bound; };
  int q = x + 1;
  const int blk_hi = min(L.n, (x / kMinBlock + 1) * kMinBlock);
  for (; q < blk_hi; ++q)
    if (hit(L.v[q])) return q;
  if (q >= L.n) return L.n;
  const int n_blk = (L.n + kMinBlock - 1) / kMinBlock;
  int blk = x / kMinBlock + 1;
  while (blk < n_blk && !hit(L.bmin[blk])) ++blk;
  if (blk >= n_blk) return L.n;
  for (q = blk * kMinBlock; q < L.n; ++q)
    if (hit(L.v[q])) return q;
  return L.n;
}
// Creating position of the interval of depth d that contains position pos (lcp[pos] >= d, d > 0).
__device__ __forceinline__ int creator_of(const Lcp& L, int pos, int d) {
  const int a = L.v[pos] < d ? pos : prev_below<true>(L, pos, d);     // (pos itself is never below d here)
  return next_below<false>(L, a, d);
}

struct TreeOut {
  int32_t *path_leaf_node, *node_parent, *node_kv_len, *node_src_path, *node_src_offset, *num_nodes;
};
struct TreeTmp {      // n + 1 entries each
  int *bmin, *c_start, *c_end, *cnt, *rank_by_pos;
};

__global__ void block_min_kernel(const int* __restrict__ lcp, int n, int* __restrict__ bmin, int* __restrict__ cnt) {
  ss::grid_dependency_enter();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t <= n) cnt[t] = 0;
  if (t >= (n + kMinBlock - 1) / kMinBlock) return;
  int m = 0x7fffffff;
  for (int i = t * kMinBlock; i < min(n, (t + 1) * kMinBlock); ++i) m = min(m, lcp[i]);
  bmin[t] = m;
}

// Marks the creating positions, finds their intervals and counts the intervals per start rank.
__global__ void creators_kernel(Lcp L, TreeTmp T) {
  ss::grid_dependency_enter();
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= L.n) return;
  const int d = L.v[x];
  int start = -1;
  if (x > 0 && d > 0) {
    const int p = prev_below<false>(L, x, d);
    if (L.v[p] < d) {                                         // no earlier position of this interval has depth d
      start = p;
      T.c_end[x] = next_below<true>(L, x, d) - 1;
      atomicAdd(&T.cnt[p], 1);
    }
  }
  T.c_start[x] = start;
}

// One block: cnt[a] (intervals that start at rank a) -> exclusive prefix sums, cnt[n] = number of inner nodes.
__global__ void scan_counts_kernel(int* __restrict__ cnt, int n, int32_t* __restrict__ num_nodes,
                                   const int32_t* __restrict__ status) {
  ss::grid_dependency_enter();
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base <= n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i <= n ? cnt[i] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
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
    const int excl = carry_s + (warp ? warp_tot[warp - 1] : 0) + incl - v;
    if (i <= n) cnt[i] = excl;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) *num_nodes = *status == SS_OK ? n + cnt[n] : 0;   // (cnt[n] had no interval: it is the total)
}

// Rank of every interval among the inner nodes in depth-first order: intervals that start earlier come first, and of
// the intervals that start at the same rank the outer ones (they end later).
__global__ void rank_kernel(Lcp L, TreeTmp T) {
  ss::grid_dependency_enter();
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= L.n) return;
  const int a = T.c_start[x];
  if (a < 0) return;
  const int floor_d = L.v[a];                                 // what the surroundings on the left share
  int outer = 0, e = T.c_end[x];
  for (;;) {                                                  // walk outwards through the intervals with the same start
    const int v = e + 1 < L.n ? L.v[e + 1] : 0;
    if (v <= floor_d) break;
    ++outer;
    e = next_below<true>(L, e + 1, v) - 1;
  }
  T.rank_by_pos[x] = T.cnt[a] + outer;
}

// Inner nodes: id, parent, length, source.  Leaves likewise.  (d pages deep <=> d * page tokens on the chain above.)
__global__ void emit_kernel(Seqs S, Lcp L, const int* __restrict__ idx, TreeTmp T, TreeOut O,
                            const int32_t* __restrict__ status) {
  ss::grid_dependency_enter();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= L.n || *status != SS_OK) return;
  // ---- the interval created at position r, if any ---------------------------------------------------------------------
  const int a = T.c_start[r];
  if (a >= 0) {
    const int d = L.v[r], e = T.c_end[r];
    const int left = L.v[a], right = e + 1 < L.n ? L.v[e + 1] : 0;
    const int id = T.rank_by_pos[r] + a;                      // `a` leaves precede it
    int parent = -1, pd = 0;
    if (right > left) {                                       // the next outer interval starts at the same rank
      parent = id - 1;
      pd = right;
    } else if (left > 0) {
      const int y = creator_of(L, a, left);
      parent = T.rank_by_pos[y] + T.c_start[y];
      pd = left;
    }
    O.node_parent[id] = parent;
    O.node_kv_len[id] = (d - pd) * S.page;
    O.node_src_path[id] = idx[a];
    O.node_src_offset[id] = pd * S.page;
  }
  // ---- the leaf of rank r ---------------------------------------------------------------------------------------------
  {
    const int left = L.v[r], right = r + 1 < L.n ? L.v[r + 1] : 0;
    const int pd = max(left, right);
    int parent = -1;
    if (pd > 0) {
      const int y = creator_of(L, left >= right ? r : r + 1, pd);
      parent = T.rank_by_pos[y] + T.c_start[y];
    }
    const int path = idx[r];
    const int id = r + T.cnt[r + 1];                          // every interval that starts at a rank <= r precedes it
    O.node_parent[id] = parent;
    O.node_kv_len[id] = static_cast<int>(S.tok_offsets[path + 1] - S.tok_offsets[path]) - pd * S.page;
    O.node_src_path[id] = path;
    O.node_src_offset[id] = pd * S.page;
    O.path_leaf_node[r] = id;
  }
}

struct Layout {
  size_t status, hashes, idx, lcp, tmp, total;
  int n_pad;
};

static Layout layout(int n, int64_t total_tok, int page) {
  Layout L;
  int n_pad = kSortChunk;
  while (n_pad < n) n_pad <<= 1;
  L.n_pad = n_pad;
  size_t off = 0;
  L.status = off; off = align_up(off + 256);
  L.hashes = off; off = align_up(off + (static_cast<size_t>(total_tok / page) + n + 2) * sizeof(uint64_t));
  L.idx = off; off = align_up(off + static_cast<size_t>(n_pad) * 4);
  L.lcp = off; off = align_up(off + static_cast<size_t>(n + 1) * 4);
  L.tmp = off; off = align_up(off + static_cast<size_t>(5) * (n + 1) * 4);
  L.total = off;
  return L;
}

}  // namespace ptree
}  // namespace ss

extern "C" int32_t ss_prefix_tree_workspace_bytes(int32_t n_paths, int64_t total_tok, int32_t page_size,
                                                  size_t* out_bytes) {
  if (n_paths < 0 || n_paths > SS_PREFIX_TREE_MAX_PATHS || total_tok < 0 || page_size < 1 || !out_bytes)
    return SS_ERR_INVALID_ARG;
  *out_bytes = ss::ptree::layout(n_paths, total_tok, page_size).total;
  return SS_OK;
}

extern "C" int32_t ss_build_prefix_tree(const int32_t* tok_ids, const int64_t* tok_offsets, int32_t n_paths,
                                        int64_t total_tok, int32_t page_size, int32_t* order_out,
                                        int32_t* path_leaf_node_out, int32_t* node_parent_out, int32_t* node_kv_len_out,
                                        int32_t* node_src_path_out, int32_t* node_src_offset_out,
                                        int32_t* num_nodes_out, void* workspace, size_t workspace_bytes, void* stream) {
  using namespace ss;
  using namespace ss::ptree;
  if (n_paths < 0 || n_paths > SS_PREFIX_TREE_MAX_PATHS || total_tok < 0 || page_size < 1) return SS_ERR_INVALID_ARG;
  if (!num_nodes_out || !workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign) return SS_ERR_INVALID_ARG;
  const Layout L = layout(n_paths, total_tok, page_size);
  if (workspace_bytes < L.total) return SS_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = as_stream(stream);
  char* ws = static_cast<char*>(workspace);
  int32_t* status = reinterpret_cast<int32_t*>(ws + L.status);
  if (cudaMemsetAsync(status, 0, 256, st) != cudaSuccess || cudaMemsetAsync(num_nodes_out, 0, sizeof(int32_t), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  if (n_paths == 0) return SS_OK;
  if (!tok_offsets || !order_out || !path_leaf_node_out || !node_parent_out || !node_kv_len_out || !node_src_path_out ||
      !node_src_offset_out || (total_tok > 0 && !tok_ids))
    return SS_ERR_INVALID_ARG;
  const int n = n_paths;
  uint64_t* hashes = reinterpret_cast<uint64_t*>(ws + L.hashes);
  int* idx = reinterpret_cast<int*>(ws + L.idx);
  int* lcp = reinterpret_cast<int*>(ws + L.lcp);
  int* tmp = reinterpret_cast<int*>(ws + L.tmp);
  const size_t stride = static_cast<size_t>(n) + 1;
  TreeTmp T{tmp, tmp + stride, tmp + 2 * stride, tmp + 3 * stride, tmp + 4 * stride};
  TreeOut O{path_leaf_node_out, node_parent_out, node_kv_len_out, node_src_path_out, node_src_offset_out, num_nodes_out};
  const Seqs S{tok_ids, tok_offsets, hashes, page_size};

  SS_LAUNCH(page_hash_kernel, (n + 7) / 8, 256, 0, st, tok_ids, tok_offsets, n, page_size, hashes);
  SS_LAUNCH(iota_kernel, (L.n_pad + 255) / 256, 256, 0, st, idx, n, L.n_pad);
  const int chunks = L.n_pad / kSortChunk;
  SS_LAUNCH(sort_chunks_kernel, chunks, kSortBlock, 0, st, S, idx, L.n_pad, 0);
  for (int size = 2 * kSortChunk; size <= L.n_pad; size <<= 1) {
    for (int stride2 = size >> 1; stride2 >= kSortChunk; stride2 >>= 1)
      SS_LAUNCH(merge_step_kernel, (L.n_pad / 2 + 255) / 256, 256, 0, st, S, idx, L.n_pad, size, stride2);
    SS_LAUNCH(sort_chunks_kernel, chunks, kSortBlock, 0, st, S, idx, L.n_pad, size);
  }
  SS_LAUNCH(neighbour_kernel, (n + 7) / 8, 256, 0, st, S, idx, n, lcp, order_out, status);
  const Lcp Lc{lcp, T.bmin, n};
  SS_LAUNCH(block_min_kernel, (n + 1 + 255) / 256, 256, 0, st, lcp, n, T.bmin, T.cnt);
  SS_LAUNCH(creators_kernel, (n + 255) / 256, 256, 0, st, Lc, T);
  SS_LAUNCH(scan_counts_kernel, 1, 1024, 0, st, T.cnt, n, num_nodes_out, status);
  SS_LAUNCH(rank_kernel, (n + 255) / 256, 256, 0, st, Lc, T);
  SS_LAUNCH(emit_kernel, (n + 255) / 256, 256, 0, st, S, Lc, idx, T, O, status);
  return SS_OK;
}
