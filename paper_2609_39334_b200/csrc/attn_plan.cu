// Device-side planner of ss_tree_attention: one block turns the tree + per-path arrays into work lists
// (tile items, leaf items), partial-slot assignments and per-path classes.  Running it on the device means
// the live path count can come straight from ss_dedup_paths without a host round trip.
#include "attn_plan.cuh"

namespace ss {
namespace attn {

constexpr int kPlanThreads = 1024;

// In-place exclusive scan of a[0..n) by the whole block; returns the total to every thread.
__device__ int block_excl_scan(int32_t* a, int n) {
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < n ? a[i] : 0;
    int x = v;
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
    }
    __syncthreads();
    const int before = carry_s + (warp ? warp_tot[warp - 1] : 0) + x - v;
    if (i < n) a[i] = before;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry_s = before + v;
    __syncthreads();
  }
  return carry_s;
}

// Block-uniform read of the status word (every thread gets the same answer, so an early return cannot leave
// part of the block waiting at a later barrier).
__device__ bool block_failed(const PlanHeader* hdr) {
  __shared__ int s_status;
  __syncthreads();
  if (threadIdx.x == 0) s_status = hdr->status;
  __syncthreads();
  return s_status != SS_OK;
}

__global__ void __launch_bounds__(kPlanThreads) plan_kernel(const Params P) {
  __shared__ int s_live, s_total_tiles, s_generic;
  PlanHeader* hdr = P.hdr;
  const int tid = threadIdx.x, nt = blockDim.x;
  if (tid == 0) {
    int live = P.num_paths;
    if (P.num_paths_dev) {
      live = *P.num_paths_dev;
      if (live < 0) live = 0;
      if (live > P.num_paths) live = P.num_paths;
    }
    s_live = live;
    s_total_tiles = 0;
    s_generic = 0;
    hdr->status = SS_OK;
    hdr->live_paths = live;
    hdr->n_dec = 0;
    hdr->n_tile_items = 0;
    hdr->n_leaf_items = 0;
    hdr->n_slots = 0;
    hdr->n_generic_rows = 0;
    hdr->tile_counter = 0;
    hdr->leaf_counter = 0;
  }
  __syncthreads();
  const int live = s_live;
  const int N = P.num_nodes;
  const bool force_generic = (P.flags & SS_FLAG_FORCE_GENERIC) != 0;

  // ---- nodes: depth and number of keys before the node ---------------------------------------------------
  for (int n = tid; n < N; n += nt) {
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
    for (int64_t i = tid; i < P.total_node_pages; i += nt) {
      const int pg = P.node_pages[i];
      if (pg < 0 || pg >= P.num_pages) set_status(&hdr->status, SS_ERR_BAD_INPUT);
    }
  }
  if (block_failed(hdr)) return;

  // ---- paths: class, kv length, membership counts of every chain node ---------------------------------------
  for (int p = tid; p < live; p += nt) {
    const int leaf = P.path_leaf_node[p];
    const int T = P.path_q_len[p];
    if (leaf < 0 || leaf >= N || T < 1 || P.q_offsets[p + 1] - P.q_offsets[p] != T || P.q_offsets[p] < 0 ||
        P.q_offsets[p + 1] > P.total_q) {
      set_status(&hdr->status, SS_ERR_BAD_INPUT);
      P.path_class[p] = kClassGeneric;
      P.path_scan[p] = 0;
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
    P.path_scan[p] = (cls == kClassDecode) ? 1 : 0;
    if (cls == kClassGeneric) atomicAdd(&s_generic, T);
    for (int a = leaf; a >= 0; a = P.node_parent[a]) {
      atomicMin(&P.node_first[a], p);
      atomicMax(&P.node_last[a], p);
      atomicAdd(&P.node_npaths[a], 1);
      if (cls == kClassDecode) atomicAdd(&P.node_ndec[a], 1);
    }
  }
  if (block_failed(hdr)) return;

  // ---- decode ranks ---------------------------------------------------------------------------------------------
  for (int p = tid; p < live; p += nt) P.path_dec_rank[p] = P.path_scan[p];
  const int n_dec = block_excl_scan(P.path_dec_rank, live);
  if (tid == 0) {
    P.path_dec_rank[live] = n_dec;
    hdr->n_dec = n_dec;
    hdr->n_generic_rows = s_generic;
    if (n_dec > P.caps.dec) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
  }
  if (block_failed(hdr)) return;
  for (int p = tid; p < live; p += nt)
    if (P.path_class[p] == kClassDecode) P.dec_tok[P.path_dec_rank[p]] = static_cast<int32_t>(P.q_offsets[p]);

  // ---- nodes: role, tiles ---------------------------------------------------------------------------------------
  const int tpt = P.tok_per_tile;
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
  const int total_tiles = s_total_tiles * P.Hkv;
  for (int n = tid; n < N; n += nt) {
    const int np = P.node_npaths[n], nd = P.node_ndec[n], len = P.node_kv_len[n];
    const int tiles = P.node_item_base[n];
    int splits = 1, own = 0, split_len = len;
    if (nd > 0 && len > 0) {
      if (tiles == 0) {
        own = ceil_div(len, kLeafChunk);             // private leaf of one decode path
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
    (void)np;
    P.node_splits[n] = splits;
    P.node_split_len[n] = split_len;
    P.node_own_slots[n] = own;
    P.node_item_base[n] = tiles * splits * P.Hkv;
  }
  __syncthreads();
  for (int n = tid; n < N; n += nt) {
    int off = 0;
    for (int a = P.node_parent[n]; a >= 0; a = P.node_parent[a]) off += P.node_own_slots[a];
    P.node_level_off[n] = off;
  }
  const int n_stacked = block_excl_scan(P.node_item_base, N);
  if (tid == 0) P.node_item_base[N] = n_stacked;

  // ---- decode paths: partial slots and leaf items ---------------------------------------------------------------
  for (int p = tid; p < live; p += nt) {
    int s = 0;
    if (P.path_class[p] == kClassDecode) {
      const int leaf = P.path_leaf_node[p];
      s = P.node_level_off[leaf] + P.node_own_slots[leaf];
    }
    P.path_scan[p] = s;
  }
  const int n_slots = block_excl_scan(P.path_scan, live);
  for (int p = tid; p < live; p += nt)
    if (P.path_class[p] == kClassDecode) P.dec_slot_base[P.path_dec_rank[p]] = P.path_scan[p];
  if (tid == 0) {
    P.dec_slot_base[n_dec] = n_slots;
    hdr->n_slots = n_slots;
    if (n_slots > P.caps.slots) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
  }
  __syncthreads();
  // leaf items
  for (int p = tid; p < live; p += nt) {
    int c = 0;
    if (P.path_class[p] == kClassDecode) {
      const int leaf = P.path_leaf_node[p];
      const bool leaf_only = (P.node_npaths[leaf] == 1);
      if (leaf_only && P.node_kv_len[leaf] > 0) c = ceil_div(P.node_kv_len[leaf], kLeafChunk) * P.Hkv;
    }
    P.path_scan[p] = c;
  }
  const int n_leaf_items = block_excl_scan(P.path_scan, live);
  if (tid == 0) {
    hdr->n_leaf_items = n_leaf_items;
    if (n_leaf_items > P.caps.leaf_items) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
  }
  if (block_failed(hdr)) return;
  for (int p = tid; p < live; p += nt) {
    if (P.path_class[p] != kClassDecode) continue;
    const int leaf = P.path_leaf_node[p];
    const int len = P.node_kv_len[leaf];
    if (!(P.node_npaths[leaf] == 1 && len > 0)) continue;
    const int chunks = ceil_div(len, kLeafChunk);
    int e = P.path_scan[p];
    const int slot0 = P.dec_slot_base[P.path_dec_rank[p]] + P.node_level_off[leaf];
    for (int c = 0; c < chunks; ++c)
      for (int g = 0; g < P.Hkv; ++g) {
        LeafItem it;
        it.q_row = static_cast<int32_t>(P.q_offsets[p]);
        it.node = leaf;
        it.g = g;
        it.kv_begin = c * kLeafChunk;
        it.kv_end = min(len, (c + 1) * kLeafChunk);
        it.slot = slot0 + c;
        it.pad0 = it.pad1 = 0;
        P.leaf_items[e++] = it;
      }
  }
  __syncthreads();

  // ---- chain paths: tile items ----------------------------------------------------------------------------------
  for (int p = tid; p < live; p += nt)
    P.path_scan[p] = (P.path_class[p] == kClassChain) ? ceil_div(P.path_q_len[p], tpt) * P.Hkv : 0;
  const int n_chain = block_excl_scan(P.path_scan, live);
  const int n_items = n_stacked + n_chain;
  if (tid == 0) {
    hdr->n_tile_items = n_items;
    if (n_items > P.caps.tile_items) set_status(&hdr->status, SS_ERR_WORKSPACE_TOO_SMALL);
  }
  if (block_failed(hdr)) return;

  // stacked items: item e -> node by binary search over the exclusive scan of per-node item counts
  for (int e = tid; e < n_stacked; e += nt) {
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
    P.tile_items[e] = it;
  }
  for (int p = tid; p < live; p += nt) {
    if (P.path_class[p] != kClassChain) continue;
    const int T = P.path_q_len[p];
    const int L = P.path_kv_len[p];
    const int tiles = ceil_div(T, tpt);
    int e = n_stacked + P.path_scan[p];
    for (int g = 0; g < P.Hkv; ++g)
      for (int t = 0; t < tiles; ++t) {
        TileItem it;
        it.node = P.path_leaf_node[p];
        it.tok0 = static_cast<int32_t>(P.q_offsets[p]) + t * tpt;
        it.n_tok = min(tpt, T - t * tpt);
        it.kind_g = (kItemChain << 16) | g;
        it.kv_begin = 0;
        it.limit0 = L - T + t * tpt + 1;
        it.kv_end = max(0, min(L, it.limit0 + it.n_tok - 1));
        it.slot_off = -1;
        P.tile_items[e++] = it;
      }
  }
}

int32_t launch_plan(const Params& P, cudaStream_t st) {
  SS_LAUNCH(plan_kernel, 1, kPlanThreads, 0, st, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
