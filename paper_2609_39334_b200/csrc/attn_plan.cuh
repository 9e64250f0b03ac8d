// Plan structures of ss_tree_attention: how the tree of candidate paths is cut into kernel work items.
//
// Path classes
//   DECODE   T == 1.  Level-split: every node on the chain that is shared (or is not this path's private
//            leaf) is processed once for ALL decode tokens below it by stacked "tile items" (tensor cores),
//            the path's private leaf by "leaf items" (bandwidth-bound kernel); the per-level partial results
//            are combined by the log-sum-exp merge.
//   CHAIN    T > 1 (a verification step).  A tile of up to 128 stacked rows (tokens x GQA group) of ONE path
//            walks the path's whole KV chain root -> leaf in one pass (causal tail inside the leaf) and writes
//            the final result: no partials.  Shared prefixes are re-used through L2.
//   GENERIC  anything the fast kernels do not take (an inner chain node that is not a whole number of pages,
//            a GQA group > 16 for decode, or SS_FLAG_FORCE_GENERIC): one warp per (query token, head).
#pragma once
#include "common.cuh"

namespace ss {
namespace attn {

constexpr int kHeadDim = 128;
constexpr int kPage = 16;
constexpr int kTileRows = 128;          // stacked rows of one tile item
constexpr int kKvTile = 64;             // keys per tensor-core step
constexpr int kLeafChunk = 256;         // most keys per leaf item (decode); small calls use 128 or 64, see Params::leaf_chunk
constexpr int kMaxRootSplits = 8;       // KV splits of a root node when there are few tiles
constexpr int kMinSplitLen = 512;       // a split is at least this many keys

enum PathClass : int32_t { kClassDecode = 0, kClassChain = 1, kClassGeneric = 2 };
enum ItemKind : int32_t { kItemStacked = 0, kItemChain = 1 };

// One tile of stacked query rows against a KV source.  40 bytes.
struct alignas(8) TileItem {
  int32_t node;       // stacked: the shared node; chain: the path's leaf node
  int32_t tok0;       // stacked: index into dec_tok[]; chain: first query row (global token index)
  int32_t n_tok;      // tokens in the tile (rows = n_tok * G)
  int32_t kind_g;     // kind << 16 | kv head
  int32_t kv_begin;   // token range [kv_begin, kv_end) of the source's virtual key sequence
  int32_t kv_end;
  int32_t limit0;     // keys visible to the tile's first token; token i sees limit0 + i * (kind == chain)
  int32_t slot_off;   // stacked: partial slot relative to the token's slot base; chain: -1 (final output)
  int32_t src0;       // chain: row of q holding the tile's first token (stacked: rows come from dec_src[])
  int32_t pad;
};

// One chunk of a decode path's private leaf.  32 bytes.
struct alignas(16) LeafItem {
  int32_t page0;      // index into node_pages of the chunk's first page
  int32_t node;       // leaf node
  int32_t g;          // kv head
  int32_t kv_begin;   // token range inside the leaf
  int32_t kv_end;
  int32_t slot;       // absolute partial slot
  int32_t q_src;      // row of q holding the token's query
  int32_t dec;        // decode rank of the token (index into dec_tok / dec_slot_base / dec_leaf_chunks)
};

struct PlanHeader {       // first bytes of the workspace; status MUST be the first word
  int32_t status;
  int32_t live_paths;
  int32_t n_dec;          // decode tokens
  int32_t n_tile_items;
  int32_t n_leaf_items;
  int32_t n_slots;
  int32_t n_generic_rows; // > 0 if any path is GENERIC
  int32_t tile_counter;   // work-stealing counters (reset by the planner)
  int32_t leaf_counter;
  int32_t n_stacked_items; // tile items [0, n_stacked_items) are stacked items, the rest chain items
  int32_t pad[6];
#ifdef SS_STAMPS
  unsigned long long stamp[40];  // instrumented build: %globaltimer at kernel starts / ends (see SS_STAMP); 8..23 (24..31: phases of the planner's scan; 32..36: of the one-block planner):
                                 // clock sums of one softmax thread per tile-kernel block (where an item's time goes)
#endif
};

// Instrumented build (-DSS_STAMPS): the first thread of a kernel records when it started (after its predecessor
// completed), every block when it ended; slots 0/1 planner, 2/3 tile kernel, 4/5 leaf kernel, 6/7 merge.
#ifdef SS_STAMPS
__device__ __forceinline__ unsigned long long ss_globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define SS_STAMP_BEGIN(hdr, i) do { if (blockIdx.x == 0 && threadIdx.x == 0) (hdr)->stamp[i] = ss_globaltimer(); } while (0)
#define SS_STAMP_END(hdr, i) do { if (threadIdx.x == 0) atomicMax(&(hdr)->stamp[i], ss_globaltimer()); } while (0)
#else
#define SS_STAMP_BEGIN(hdr, i) do { } while (0)
#define SS_STAMP_END(hdr, i) do { } while (0)
#endif

struct Caps {             // host-computed capacities of the plan arrays
  int32_t dec, tile_items, leaf_items;
  int64_t slots;
};

// Everything a kernel needs, passed by value.
struct Params {
  int32_t Hq, Hkv, G, tok_per_tile;
  float scale, scale_log2;
  uint32_t flags;
  const __nv_bfloat16 *k_pool, *v_pool;
  int64_t num_pages, page_stride, head_stride, token_stride;
  int32_t num_nodes;
  const int32_t *node_parent, *node_kv_len;
  const int64_t* node_page_offsets;
  const int32_t* node_pages;
  int64_t total_node_pages;
  int32_t num_paths;
  const int32_t *num_paths_dev, *path_leaf_node, *path_q_len;
  const int64_t* q_offsets;
  const int64_t* q_src_offsets;  // optional: where each path's query rows start inside q
  int64_t q_src_rows;
  int64_t total_q;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  float* lse;
  int32_t target_tiles;      // the planner splits root nodes until about this many tile items exist
  int32_t leaf_chunk;        // keys per leaf item: 256, or less when the call is too small to keep every warp of the
                             // leaf kernel supplied with several items (chosen on the host from the page count)
  Caps caps;
  // ---- workspace regions ----
  PlanHeader* hdr;
  int32_t *node_start, *node_depth, *node_first, *node_last, *node_npaths, *node_ndec, *node_own_slots,
      *node_level_off, *node_item_base, *node_splits, *node_split_len;
  int32_t *path_class, *path_kv_len, *path_dec_rank, *path_slot_base, *path_leaf_base, *path_chain_base;
  int32_t *dec_tok, *dec_src, *dec_slot_base;   // per decode token: output row, query row, first partial slot
  int32_t *dec_leaf_chunks;  // per decode token: leaf items per kv head (0: empty or shared leaf)
  int32_t *leaf_arrive;      // [decode token][kv head]: leaf items that have written their partial (zeroed by the planner)
  TileItem* tile_items;
  LeafItem* leaf_items;
  float* part_o;             // [slots][Hq][128]
  float* part_lse;           // [slots][Hq]
};

}  // namespace attn
}  // namespace ss
