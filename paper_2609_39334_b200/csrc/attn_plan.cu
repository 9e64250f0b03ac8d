// Device-side planner of ss_tree_attention: turns the tree + per-path arrays into work lists (tile items, leaf
// items), partial-slot assignments and per-path classes.  Running it on the device means the live path count can
// come straight from ss_dedup_paths without a host round trip.  Four phases:
//   nodes   depth and prefix length of every node, range checks, counters reset
//   paths   class and key length of every path, membership counts of its chain nodes
//   scan    (one block) every prefix sum: decode ranks, per-node tile items and KV splits, partial slots, leaf
//           items, chain items; capacity checks; totals into the header
//   emit    writes the item lists and the per-decode-token arrays
// Trees of up to kSmallPlan nodes and paths (every benchmark configuration but the largest) are planned by ONE
// block in ONE launch: the tree arrays and all intermediate arrays live in shared memory (the phase functions only
// see redirected pointers), so the whole plan costs three or four round trips to global memory instead of the
// dozens that the dependent loads and in-place scans of the general path make.  Larger inputs take four launches
// (nodes, paths and emit grid-parallel, scan in one block).
// The header (status word first) is cleared by the host-side launcher before the first of the four kernels; the
// one-block planner builds it in shared memory and writes it out whole.
#include "attn_plan.cuh"

namespace ss {
namespace attn {

constexpr int kScanThreads = 1024;
constexpr int kGridThreads = 256;

// In-place exclusive scan of a[0..n) by one whole block: every thread sums a contiguous chunk, the chunk sums are
// scanned across the block, then every thread rewrites its chunk.  Returns the total to every thread.
__device__ int block_excl_scan_chunks(int32_t* a, int n) {
  __shared__ int warp_tot[32];
  __shared__ int total_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int chunk = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min(n, static_cast<int>(threadIdx.x) * chunk), hi = min(n, lo + chunk);
  __syncthreads();
  int sum = 0;
  for (int i = lo; i < hi; ++i) sum += a[i];
  int x = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) warp_tot[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int t = lane < nw ? warp_tot[lane] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, t, o);
      if (lane >= o) t += y;
    }
    warp_tot[lane] = t;
    if (lane == 31) total_s = t;
  }
  __syncthreads();
  int run = (warp ? warp_tot[warp - 1] : 0) + x - sum;
  for (int i = lo; i < hi; ++i) {
    const int v = a[i];
    a[i] = run;
    run += v;
  }
  __syncthreads();
  return total_s;
}

// Four independent scans of equal length in one pass (same scheme, one set of barriers): for the per-path arrays of
// the one-block planner, where a scan is three barrier round trips and little else.
__device__ void block_excl_scan4_chunks(int32_t* a0, int32_t* a1, int32_t* a2, int32_t* a3, int n, int (&total)[4]) {
  __shared__ int warp_tot4[32][4];
  __shared__ int total4_s[4];
  int32_t* a[4] = {a0, a1, a2, a3};
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int chunk = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min(n, static_cast<int>(threadIdx.x) * chunk), hi = min(n, lo + chunk);
  __syncthreads();
  int sum[4], x[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    sum[k] = 0;
    for (int i = lo; i < hi; ++i) sum[k] += a[k][i];
    x[k] = sum[k];
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int y = __shfl_up_sync(0xffffffffu, x[k], o);
      if (lane >= o) x[k] += y;
    }
  }
  if (lane == 31) {
#pragma unroll
    for (int k = 0; k < 4; ++k) warp_tot4[warp][k] = x[k];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      int t = lane < nw ? warp_tot4[lane][k] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      warp_tot4[lane][k] = t;
      if (lane == 31) total4_s[k] = t;
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    int run = (warp ? warp_tot4[warp - 1][k] : 0) + x[k] - sum[k];
    for (int i = lo; i < hi; ++i) {
      const int v = a[k][i];
      a[k][i] = run;
      run += v;
    }
    total[k] = total4_s[k];
  }
  __syncthreads();
}

// The same for arrays in GLOBAL memory of up to 16 entries per thread: a thread keeps its 16 consecutive entries of
// each array in registers (128-bit loads, all issued before the first is used; 128-bit stores), so a pair of scans
// costs two trips to memory instead of the six of two staged scans.  The arrays must be 16-byte aligned.
constexpr int kScanRegs = 16;
__device__ void block_excl_scan2_regs(int32_t* a0, int32_t* a1, int n, int (&total)[2]) {   // (two arrays per call: 32 of a thread's 64 registers)
  __shared__ int warp_tot4[32][2];
  __shared__ int total4_s[2];
  int32_t* a[2] = {a0, a1};
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int lo = static_cast<int>(threadIdx.x) * kScanRegs;
  int v[2][kScanRegs];
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 2; ++k) {
#pragma unroll
    for (int i = 0; i < kScanRegs; i += 4) {
      if (lo + i + 4 <= n) {
        const int4 q = *reinterpret_cast<const int4*>(a[k] + lo + i);
        v[k][i] = q.x; v[k][i + 1] = q.y; v[k][i + 2] = q.z; v[k][i + 3] = q.w;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[k][i + j] = (lo + i + j < n) ? a[k][lo + i + j] : 0;
      }
    }
  }
  int sum[2], x[2];
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    sum[k] = 0;
#pragma unroll
    for (int i = 0; i < kScanRegs; ++i) sum[k] += v[k][i];
    x[k] = sum[k];
  }
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int y = __shfl_up_sync(0xffffffffu, x[k], o);
      if (lane >= o) x[k] += y;
    }
  }
  if (lane == 31) {
#pragma unroll
    for (int k = 0; k < 2; ++k) warp_tot4[warp][k] = x[k];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      int t = lane < nw ? warp_tot4[lane][k] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) t += y;
      }
      warp_tot4[lane][k] = t;
      if (lane == 31) total4_s[k] = t;
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    int run = (warp ? warp_tot4[warp - 1][k] : 0) + x[k] - sum[k];
#pragma unroll
    for (int i = 0; i < kScanRegs; i += 4) {
      int4 q;
      q.x = run; run += v[k][i];
      q.y = run; run += v[k][i + 1];
      q.z = run; run += v[k][i + 2];
      q.w = run; run += v[k][i + 3];
      if (lo + i + 4 <= n) {
        *reinterpret_cast<int4*>(a[k] + lo + i) = q;
      } else {
        if (lo + i < n) a[k][lo + i] = q.x;
        if (lo + i + 1 < n) a[k][lo + i + 1] = q.y;
        if (lo + i + 2 < n) a[k][lo + i + 2] = q.z;
      }
    }
    total[k] = total4_s[k];
  }
  __syncthreads();
}

// The same scan for an array in GLOBAL memory: it goes through the block's staging buffer in shared memory when it
// fits (coalesced in, scanned on chip, coalesced out) - every thread walking its own contiguous chunk of a global
// array makes each load touch 32 different sectors, which cost the one-block scan kernel most of its time.
constexpr int kScanStage = 16384;                  // entries of the staging buffer (64 KB, dynamic shared memory)
__device__ int block_excl_scan(int32_t* a, int n, int32_t* stage) {
  if (stage == nullptr || n > kScanStage) return block_excl_scan_chunks(a, n);
  __syncthreads();
  for (int i = threadIdx.x; i < n; i += blockDim.x) stage[i] = a[i];
  const int total = block_excl_scan_chunks(stage, n);      // (starts and ends with a barrier)
  for (int i = threadIdx.x; i < n; i += blockDim.x) a[i] = stage[i];
  __syncthreads();
  return total;
}

// Block-uniform read of the status word (every thread gets the same answer, so an early return cannot leave
// part of the block waiting at a later barrier).
__device__ bool block_failed(const PlanHeader* hdr) {
  __shared__ int s_status;
  __syncthreads();
  if (threadIdx.x == 0) s_status = *reinterpret_cast<const volatile int32_t*>(&hdr->status);
  __syncthreads();
  return s_status != SS_OK;
}

__device__ __forceinline__ int live_paths(const Params& P) {
  int live = P.num_paths;
  if (P.num_paths_dev) {
    live = *P.num_paths_dev;
    if (live < 0) live = 0;
    if (live > P.num_paths) live = P.num_paths;
  }
  return live;
}

// ---- nodes: depth and number of keys before the node -------------------------------------------------------------
__device__ __forceinline__ void plan_nodes_phase(const Params& P) {
  PlanHeader* hdr = P.hdr;
  const int64_t gtid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t gsize = static_cast<int64_t>(gridDim.x) * blockDim.x;
  if (gtid == 0) hdr->live_paths = live_paths(P);
  for (int64_t n64 = gtid; n64 < P.num_nodes; n64 += gsize) {
    const int n = static_cast<int>(n64);
    int d = 0, start = 0;
    int a = P.node_parent[n];
    bool bad = (a >= n || a < -1 || P.node_kv_len[n] < 0);
    while (!bad && a >= 0 && d < SS_MAX_DEPTH) {
      start += P.node_kv_len[a];
      ++d;
      const int na = P.node_parent[a];
      if (na >= a || na < -1) { bad = true; break; }
      a = na;
    }
    if (bad) set_status(&hdr->status, SS_ERR_BAD_INPUT);
    else if (a >= 0 || d + 1 > SS_MAX_DEPTH) set_status(&hdr->status, SS_ERR_UNSUPPORTED);
    const int64_t np = P.node_page_offsets[n + 1] - P.node_page_offsets[n];
    if (!bad && (np < 0 || np * kPage < P.node_kv_len[n] || P.node_page_offsets[n + 1] > P.total_node_pages ||
                 P.node_page_offsets[n] < 0))
      set_status(&hdr->status, SS_ERR_BAD_INPUT);
    P.node_depth[n] = d;
    P.node_start[n] = start;
    P.node_first[n] = 0x7fffffff;
    P.node_last[n] = -1;
    P.node_npaths[n] = 0;
    P.node_ndec[n] = 0;
  }
  if (P.flags & SS_FLAG_VALIDATE) {
    for (int64_t i = gtid; i < P.total_node_pages; i += gsize) {
      const int pg = P.node_pages[i];
      if (pg < 0 || pg >= P.num_pages) set_status(&hdr->status, SS_ERR_BAD_INPUT);
    }
  }
}

// ---- paths: class, kv length, membership counts of every chain node ------------------------------------------------
__device__ __forceinline__ void plan_paths_phase(const Params& P) {
  PlanHeader* hdr = P.hdr;
  const int live = live_paths(P);
  const int N = P.num_nodes;
  const bool force_generic = (P.flags & SS_FLAG_FORCE_GENERIC) != 0;
  const int64_t gsize = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t p64 = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p64 < live; p64 += gsize) {
    const int p = static_cast<int>(p64);
    const int leaf = P.path_leaf_node[p];
    const int T = P.path_q_len[p];
    bool bad_src = false;
    if (P.q_src_offsets) {
      const int64_t s0 = P.q_src_offsets[p];
      bad_src = s0 < 0 || s0 + T > P.q_src_rows || s0 + T > 0x7fffffffLL;
    }
    if (leaf < 0 || leaf >= N || T < 1 || P.q_offsets[p + 1] - P.q_offsets[p] != T || P.q_offsets[p] < 0 ||
        P.q_offsets[p + 1] > P.total_q || bad_src) {
      set_status(&hdr->status, SS_ERR_BAD_INPUT);
      P.path_class[p] = kClassGeneric;
      continue;
    }
    bool inner_whole_pages = true;
    for (int a = P.node_parent[leaf]; a >= 0; a = P.node_parent[a])
      if (P.node_kv_len[a] % kPage) inner_whole_pages = false;
    int cls;
    if (force_generic) cls = kClassGeneric;
    else if (T == 1) cls = (P.G <= 16) ? kClassDecode : kClassGeneric;
    else cls = inner_whole_pages ? kClassChain : kClassGeneric;
    P.path_class[p] = cls;
    P.path_kv_len[p] = P.node_start[leaf] + P.node_kv_len[leaf];
    if (cls == kClassGeneric) atomicAdd(&hdr->n_generic_rows, T);
    for (int a = leaf; a >= 0; a = P.node_parent[a]) {
      atomicMin(&P.node_first[a], p);
      atomicMax(&P.node_last[a], p);
      atomicAdd(&P.node_npaths[a], 1);
      if (cls == kClassDecode) atomicAdd(&P.node_ndec[a], 1);
    }
  }
}

// ---- every prefix sum -------------------------------------------------------------------------------------------------
__device__ __forceinline__ void plan_scan_phase(const Params& P, int32_t* stage) {   // one whole block; block-uniform
                                                                                     // returns only; stage: see block_excl_scan
  __shared__ int s_total_tiles;
  PlanHeader* hdr = P.hdr;
  if (block_failed(hdr)) return;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int live = live_paths(P);
  const int N = P.num_nodes;
  const int tpt = P.tok_per_tile;
  if (tid == 0) s_total_tiles = 0;

#ifdef SS_STAMPS
  long long pt = clock64();
  int pi = 24;
#define PLAN_MARK() do { __syncthreads(); if (tid == 0) { const long long t = clock64(); hdr->stamp[pi] = t - pt; pt = t; } ++pi; } while (0)
#else
#define PLAN_MARK() do { } while (0)
#endif
  // decode ranks (scanned together with the per-path counts below where one pass can take all four arrays)
  const bool fused_regs = stage != nullptr && live <= nt * kScanRegs &&
                          ((reinterpret_cast<uintptr_t>(P.path_slot_base) | reinterpret_cast<uintptr_t>(P.path_leaf_base) |
                            reinterpret_cast<uintptr_t>(P.path_chain_base) | reinterpret_cast<uintptr_t>(P.path_dec_rank)) & 15) == 0;
  const bool fused = stage == nullptr || fused_regs;
  for (int p = tid; p < live; p += nt) P.path_dec_rank[p] = (P.path_class[p] == kClassDecode) ? 1 : 0;
  if (!fused) {
    const int n_dec = block_excl_scan(P.path_dec_rank, live, stage);
    if (tid == 0) {
      P.path_dec_rank[live] = n_dec;
      hdr->n_dec = n_dec;
      if (n_dec > P.caps.dec) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
    }
  }

  PLAN_MARK();   // 8: decode ranks
  // nodes: role, tiles
  for (int n = tid; n < N; n += nt) {
    const int np = P.node_npaths[n];
    if (np > 0 && P.node_last[n] - P.node_first[n] + 1 != np) set_status(&hdr->status, SS_ERR_BAD_INPUT);
    const int nd = P.node_ndec[n], len = P.node_kv_len[n];
    int tiles = 0;
    if (nd > 0 && len > 0) {
      const bool leaf_only = (np == 1 && P.path_leaf_node[P.node_first[n]] == n);
      if (!leaf_only) tiles = ceil_div(nd, tpt);
    }
    P.node_item_base[n] = tiles;                     // tiles for now; becomes the item base after the scan
    if (tiles) atomicAdd(&s_total_tiles, tiles);
  }
  if (block_failed(hdr)) return;
  PLAN_MARK();   // 9: node tiles
  const int total_tiles = s_total_tiles * P.Hkv;
  for (int n = tid; n < N; n += nt) {
    const int nd = P.node_ndec[n], len = P.node_kv_len[n];
    const int tiles = P.node_item_base[n];
    int splits = 1, own = 0, split_len = len;
    if (nd > 0 && len > 0) {
      if (tiles == 0) {
        own = ceil_div(len, P.leaf_chunk);             // private leaf of one decode path
      } else {
        if (P.node_depth[n] == 0 && total_tiles < P.target_tiles) {
          int want = ceil_div(P.target_tiles, total_tiles);
          int most = len / kMinSplitLen;
          if (most > kMaxRootSplits) most = kMaxRootSplits;
          if (want > most) want = most;
          if (want > 1) {
            split_len = ceil_div(ceil_div(len, want), kKvTile) * kKvTile;
            splits = ceil_div(len, split_len);
          }
        }
        own = splits;
      }
    }
    P.node_splits[n] = splits;
    P.node_split_len[n] = split_len;
    P.node_own_slots[n] = own;
    P.node_item_base[n] = tiles * splits * P.Hkv;
  }
  __syncthreads();
  PLAN_MARK();   // 10: splits
  for (int n = tid; n < N; n += nt) {
    int off = 0;
    for (int a = P.node_parent[n]; a >= 0; a = P.node_parent[a]) off += P.node_own_slots[a];
    P.node_level_off[n] = off;
  }
  PLAN_MARK();   // 11: level offsets
  const int n_stacked = block_excl_scan(P.node_item_base, N, stage);
  PLAN_MARK();   // 12: item base scan
  if (tid == 0) P.node_item_base[N] = n_stacked;

  // decode paths: partial slots, leaf items; chain paths: tile items
  for (int p = tid; p < live; p += nt) {
    int slots = 0, leaf_items = 0, chain_items = 0;
    const int cls = P.path_class[p];
    if (cls == kClassDecode) {
      const int leaf = P.path_leaf_node[p];
      slots = P.node_level_off[leaf] + P.node_own_slots[leaf];
      if (P.node_npaths[leaf] == 1 && P.node_kv_len[leaf] > 0)
        leaf_items = ceil_div(P.node_kv_len[leaf], P.leaf_chunk) * P.Hkv;
    } else if (cls == kClassChain) {
      chain_items = ceil_div(P.path_q_len[p], tpt) * P.Hkv;
    }
    P.path_slot_base[p] = slots;
    P.path_leaf_base[p] = leaf_items;
    P.path_chain_base[p] = chain_items;
  }
  PLAN_MARK();   // 13: per-path counts
  int n_slots, n_leaf_items, n_chain;
  if (fused) {
    int tot[4];
    if (fused_regs) {
      int t2[2];
      block_excl_scan2_regs(P.path_slot_base, P.path_leaf_base, live, t2);
      tot[0] = t2[0];
      tot[1] = t2[1];
      block_excl_scan2_regs(P.path_chain_base, P.path_dec_rank, live, t2);
      tot[2] = t2[0];
      tot[3] = t2[1];
    } else block_excl_scan4_chunks(P.path_slot_base, P.path_leaf_base, P.path_chain_base, P.path_dec_rank, live, tot);
    n_slots = tot[0];
    n_leaf_items = tot[1];
    n_chain = tot[2];
    if (tid == 0) {
      P.path_dec_rank[live] = tot[3];
      hdr->n_dec = tot[3];
      if (tot[3] > P.caps.dec) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
    }
  } else {
    n_slots = block_excl_scan(P.path_slot_base, live, stage);
    n_leaf_items = block_excl_scan(P.path_leaf_base, live, stage);
    n_chain = block_excl_scan(P.path_chain_base, live, stage);
  }
  PLAN_MARK();   // 14: three scans
  if (tid == 0) {
    hdr->n_slots = n_slots;
    hdr->n_stacked_items = n_stacked;
    if (n_slots > P.caps.slots || n_leaf_items > P.caps.leaf_items || n_stacked + n_chain > P.caps.tile_items) {
      set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);     // the executors see the status and do nothing
    } else {
      hdr->n_leaf_items = n_leaf_items;
      hdr->n_tile_items = n_stacked + n_chain;
    }
  }
}

// ---- item lists ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void plan_emit_phase(const Params& P) {
  PlanHeader* hdr = P.hdr;
  const int live = live_paths(P);
  const int N = P.num_nodes;
  const int tpt = P.tok_per_tile;
  const int n_stacked = hdr->n_stacked_items;
  const int64_t gtid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t gsize = static_cast<int64_t>(gridDim.x) * blockDim.x;
  if (gtid == 0) P.dec_slot_base[hdr->n_dec] = hdr->n_slots;

  // per decode token: output row, query row, partial slots, leaf chunks, arrival counters
  for (int64_t p64 = gtid; p64 < live; p64 += gsize) {
    const int p = static_cast<int>(p64);
    if (P.path_class[p] != kClassDecode) continue;
    const int rank = P.path_dec_rank[p];
    const int leaf = P.path_leaf_node[p];
    const int len = P.node_kv_len[leaf];
    P.dec_tok[rank] = static_cast<int32_t>(P.q_offsets[p]);
    P.dec_src[rank] = static_cast<int32_t>(P.q_src_offsets ? P.q_src_offsets[p] : P.q_offsets[p]);
    P.dec_slot_base[rank] = P.path_slot_base[p];
    const bool own_leaf = P.node_npaths[leaf] == 1 && len > 0;
    P.dec_leaf_chunks[rank] = own_leaf ? ceil_div(len, P.leaf_chunk) : 0;
    for (int g = 0; g < P.Hkv; ++g) P.leaf_arrive[static_cast<int64_t>(rank) * P.Hkv + g] = 0;
  }
  // Leaf and chain items, one thread per ITEM (consecutive threads write consecutive descriptors: a thread per path
  // writing its own run of descriptors makes every store instruction touch 32 different sectors, and that alone cost
  // tens of microseconds on one SM).  Item e -> path by binary search over the exclusive scans.
  auto path_of = [&](const int32_t* base, int e) {
    int lo = 0, hi = live;                    // last p with base[p] <= e (paths without items share their successor's base)
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (base[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
  };
  const int n_leaf_items = hdr->n_leaf_items;
  for (int64_t e64 = gtid; e64 < n_leaf_items; e64 += gsize) {
    const int e = static_cast<int>(e64);
    const int p = path_of(P.path_leaf_base, e);
    const int local = e - P.path_leaf_base[p];
    const int c = local / P.Hkv, g = local - c * P.Hkv;
    const int leaf = P.path_leaf_node[p];
    const int len = P.node_kv_len[leaf];
    LeafItem it;
    it.page0 = static_cast<int32_t>(P.node_page_offsets[leaf]) + c * (P.leaf_chunk / kPage);
    it.node = leaf;
    it.g = g;
    it.kv_begin = c * P.leaf_chunk;
    it.kv_end = min(len, (c + 1) * P.leaf_chunk);
    it.slot = P.path_slot_base[p] + P.node_level_off[leaf] + c;
    it.q_src = static_cast<int32_t>(P.q_src_offsets ? P.q_src_offsets[p] : P.q_offsets[p]);
    it.dec = P.path_dec_rank[p];
    P.leaf_items[e] = it;
  }
  const int n_chain_items = hdr->n_tile_items - n_stacked;
  for (int64_t e64 = gtid; e64 < n_chain_items; e64 += gsize) {
    const int e = static_cast<int>(e64);
    const int p = path_of(P.path_chain_base, e);
    const int local = e - P.path_chain_base[p];
    const int T = P.path_q_len[p];
    const int L = P.path_kv_len[p];
    const int tiles = ceil_div(T, tpt);
    const int g = local / tiles, t = local - g * tiles;
    const int32_t src_row = static_cast<int32_t>(P.q_src_offsets ? P.q_src_offsets[p] : P.q_offsets[p]);
    TileItem it;
    it.node = P.path_leaf_node[p];
    it.tok0 = static_cast<int32_t>(P.q_offsets[p]) + t * tpt;
    it.n_tok = min(tpt, T - t * tpt);
    it.kind_g = (kItemChain << 16) | g;
    it.kv_begin = 0;
    it.limit0 = L - T + t * tpt + 1;
    it.kv_end = max(0, min(L, it.limit0 + it.n_tok - 1));
    it.slot_off = -1;
    it.src0 = src_row + t * tpt;
    it.pad = 0;
    P.tile_items[n_stacked + e] = it;
  }

  // stacked items: item e -> node by binary search over the exclusive scan of per-node item counts
  for (int64_t e64 = gtid; e64 < n_stacked; e64 += gsize) {
    const int e = static_cast<int>(e64);
    int lo = 0, hi = N;                       // last n with base[n] <= e and base[n+1] > e
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (P.node_item_base[mid] <= e) lo = mid; else hi = mid;
    }
    const int n = lo;
    const int local = e - P.node_item_base[n];
    const int splits = P.node_splits[n];
    const int split = local % splits;
    const int rest = local / splits;
    const int g = rest % P.Hkv;
    const int tile = rest / P.Hkv;
    const int len = P.node_kv_len[n];
    const int split_len = P.node_split_len[n];
    const int nd = P.node_ndec[n];
    TileItem it;
    it.node = n;
    it.tok0 = P.path_dec_rank[P.node_first[n]] + tile * tpt;
    it.n_tok = min(tpt, nd - tile * tpt);
    it.kind_g = (kItemStacked << 16) | g;
    it.kv_begin = split * split_len;
    it.kv_end = min(len, (split + 1) * split_len);
    it.limit0 = it.kv_end;
    it.slot_off = P.node_level_off[n] + split;
    it.src0 = 0;
    it.pad = 0;
    P.tile_items[e] = it;
  }
}

// ---- general path: four launches ------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kGridThreads) plan_nodes_kernel(const Params P) {
  ss::grid_dependency_enter();
  plan_nodes_phase(P);
}
__global__ void __launch_bounds__(kGridThreads) plan_paths_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;          // no barrier in this kernel: a per-thread return is safe
  plan_paths_phase(P);
}
__global__ void __launch_bounds__(kScanThreads) plan_scan_kernel(const Params P) {
  ss::grid_dependency_enter();
  extern __shared__ __align__(16) int32_t scan_stage[];
  plan_scan_phase(P, scan_stage);
}
__global__ void __launch_bounds__(kGridThreads) plan_emit_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;          // no barrier in this kernel
  plan_emit_phase(P);
}

// ---- small trees: one block, everything in shared memory -------------------------------------------------------------
constexpr int kSmallPlan = 2048;               // nodes and paths
constexpr int kSmallNodeArrays = 11, kSmallPathArrays = 6;
// bytes of shared memory for N nodes and NP paths: staged inputs + redirected plan arrays
inline size_t small_plan_smem(int N, int NP) {
  return static_cast<size_t>(N + 1) * (8 + 4 + 4 + 4 * kSmallNodeArrays) + static_cast<size_t>(NP + 1) * (8 + 8 + 4 + 4 + 4 * kSmallPathArrays) + 64;
}

__global__ void __launch_bounds__(kScanThreads) plan_small_kernel(const Params P0) {
  ss::grid_dependency_enter();
  extern __shared__ __align__(16) uint8_t plan_smem[];
  __shared__ PlanHeader s_hdr;       // the header is built here too and written out once, at the end
  __shared__ int s_live;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int N = P0.num_nodes, NP = P0.num_paths;
  Params P = P0;
  for (int x = tid; x < static_cast<int>(sizeof(PlanHeader) / 4); x += nt) reinterpret_cast<int32_t*>(&s_hdr)[x] = 0;
  if (tid == 0) s_live = live_paths(P0);
  P.hdr = &s_hdr;
  P.num_paths_dev = &s_live;
  __syncthreads();
  SS_STAMP_BEGIN(P.hdr, 0);
  // carve: the 8-byte arrays first, then 4-byte arrays of N + 1 and of NP + 1 entries
  int64_t* s_page_off = reinterpret_cast<int64_t*>(plan_smem);
  int64_t* s_q_off = s_page_off + (N + 1);
  int64_t* s_q_src = s_q_off + (NP + 1);
  int32_t* w = reinterpret_cast<int32_t*>(s_q_src + (NP + 1));
  auto take = [&](int n) { int32_t* p = w; w += n; return p; };
  int32_t* s_parent = take(N + 1);
  int32_t* s_len = take(N + 1);
  int32_t** node_arrays[kSmallNodeArrays] = {&P.node_start, &P.node_depth, &P.node_first, &P.node_last, &P.node_npaths,
                                             &P.node_ndec, &P.node_own_slots, &P.node_level_off, &P.node_item_base,
                                             &P.node_splits, &P.node_split_len};
  for (int i = 0; i < kSmallNodeArrays; ++i) *node_arrays[i] = take(N + 1);
  int32_t* s_leaf = take(NP + 1);
  int32_t* s_qlen = take(NP + 1);
  int32_t** path_arrays[kSmallPathArrays] = {&P.path_class, &P.path_kv_len, &P.path_dec_rank, &P.path_slot_base,
                                             &P.path_leaf_base, &P.path_chain_base};
  for (int i = 0; i < kSmallPathArrays; ++i) *path_arrays[i] = take(NP + 1);
  // stage the tree and the per-path arrays (one round trip; every later chain walk stays on chip)
  for (int n = tid; n < N; n += nt) { s_parent[n] = P0.node_parent[n]; s_len[n] = P0.node_kv_len[n]; }
  for (int n = tid; n <= N; n += nt) s_page_off[n] = P0.node_page_offsets[n];
  const int live = s_live;
  for (int p = tid; p < live; p += nt) { s_leaf[p] = P0.path_leaf_node[p]; s_qlen[p] = P0.path_q_len[p]; }
  // (the row offsets too: the emission reads them per ITEM, and a global load behind each binary search was half of
  //  its time)
  for (int p = tid; p <= live; p += nt) s_q_off[p] = P0.q_offsets[p];
  if (P0.q_src_offsets) {
    for (int p = tid; p < live; p += nt) s_q_src[p] = P0.q_src_offsets[p];
    P.q_src_offsets = s_q_src;
  }
  P.q_offsets = s_q_off;
  P.node_parent = s_parent;
  P.node_kv_len = s_len;
  P.node_page_offsets = s_page_off;
  P.path_leaf_node = s_leaf;
  P.path_q_len = s_qlen;
  __syncthreads();

#ifdef SS_STAMPS
  long long small_t = clock64();
#define SMALL_MARK(i) do { __syncthreads(); if (tid == 0) { const long long t = clock64(); s_hdr.stamp[i] = t - small_t; small_t = t; } } while (0)
#else
#define SMALL_MARK(i) do { } while (0)
#endif
  SMALL_MARK(32);                                    // staging of the inputs
  plan_nodes_phase(P);
  bool failed = block_failed(P.hdr);
  SMALL_MARK(33);
  if (!failed) {
    plan_paths_phase(P);
    __syncthreads();
    SMALL_MARK(34);
    plan_scan_phase(P, nullptr);                     // (the arrays are in shared memory already)
    failed = block_failed(P.hdr);
    SMALL_MARK(35);
  }
  if (!failed) {
    plan_emit_phase(P);
    SMALL_MARK(36);
    // the executors read these three from the workspace (exact second pass, generic rows)
    for (int n = tid; n < N; n += nt) P0.node_start[n] = P.node_start[n];
    for (int p = tid; p < live; p += nt) { P0.path_class[p] = P.path_class[p]; P0.path_kv_len[p] = P.path_kv_len[p]; }
  }
  SS_STAMP_END(P.hdr, 1);
  __syncthreads();
  for (int x = tid; x < static_cast<int>(sizeof(PlanHeader) / 4); x += nt)
    reinterpret_cast<int32_t*>(P0.hdr)[x] = reinterpret_cast<const int32_t*>(&s_hdr)[x];
}

int32_t launch_plan(const Params& P, cudaStream_t st) {
  if (P.num_nodes <= kSmallPlan && P.num_paths <= kSmallPlan) {     // (this kernel writes the whole header itself)
    static bool configured[kDeviceSlots] = {false};
    const int dev_slot = current_device_slot();
    if (dev_slot < 0 || !configured[dev_slot]) {
      if (cudaFuncSetAttribute(plan_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               static_cast<int>(small_plan_smem(kSmallPlan, kSmallPlan))) != cudaSuccess) {
        (void)cudaGetLastError();
        return SS_ERR_CUDA;
      }
      if (dev_slot >= 0) configured[dev_slot] = true;
    }
    SS_LAUNCH(plan_small_kernel, 1, kScanThreads, small_plan_smem(P.num_nodes, P.num_paths), st, P);
    return SS_OK;
  }
  if (cudaMemsetAsync(P.hdr, 0, sizeof(PlanHeader), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  const int64_t work = P.num_nodes > P.num_paths ? P.num_nodes : P.num_paths;
  int blocks = static_cast<int>((work + kGridThreads - 1) / kGridThreads);
  if (blocks < 1) blocks = 1;
  if (blocks > 1184) blocks = 1184;
  SS_LAUNCH(plan_nodes_kernel, blocks, kGridThreads, 0, st, P);
  SS_LAUNCH(plan_paths_kernel, blocks, kGridThreads, 0, st, P);
  {
    static bool configured[kDeviceSlots] = {false};
    const int dev_slot = current_device_slot();
    if (dev_slot < 0 || !configured[dev_slot]) {
      if (cudaFuncSetAttribute(plan_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kScanStage * 4) != cudaSuccess) {
        (void)cudaGetLastError();
        return SS_ERR_CUDA;
      }
      if (dev_slot >= 0) configured[dev_slot] = true;
    }
  }
  SS_LAUNCH(plan_scan_kernel, 1, kScanThreads, kScanStage * 4, st, P);
  // one thread per ITEM (there are an order of magnitude more items than paths; their number is known on the device
  // only): a grid that covers the typical item count in one or two strides
  SS_LAUNCH(plan_emit_kernel, blocks < 64 ? 8 * blocks : 1184, kGridThreads, 0, st, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
