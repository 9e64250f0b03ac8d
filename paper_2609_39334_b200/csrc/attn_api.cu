// ss_tree_attention: host side.  Checks the descriptor, lays the plan arrays out in the caller's workspace,
// and enqueues   plan -> { tile items (tcgen05) | leaf items | generic rows } -> merge   on the caller's stream.
#include <math.h>
#include <string.h>

#include "attn_plan.cuh"

namespace ss {
namespace attn {

int32_t launch_plan(const Params& P, cudaStream_t st);
int32_t launch_generic(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_tile_items_simple(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_leaf_items_simple(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_merge(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_leaf_items(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_tile_items_umma(const Params& P, cudaStream_t st, int sm_count);
int32_t launch_tile_items_umma_split(const Params& P, cudaStream_t st, int sm_count);
bool leaf_stream_supported(const Params& P);
int32_t launch_leaf_stream(const Params& P, cudaStream_t st, int sm_count);

// ---- per-phase event timing (diagnostics) ------------------------------------------------------------------
constexpr int kProfCalls = 256;                      // timed calls between two reads
struct Profiler {
  bool on = false;
  bool created = false;
  int used = 0;                                      // timed calls recorded
  cudaEvent_t ev[kProfCalls][SS_NUM_PHASES + 1];
  bool ran[kProfCalls][SS_NUM_PHASES];
};
static Profiler g_prof;

static bool prof_begin_call() {
  if (!g_prof.on || g_prof.used >= kProfCalls) return false;
  if (!g_prof.created) {
    for (int c = 0; c < kProfCalls; ++c)
      for (int e = 0; e <= SS_NUM_PHASES; ++e)
        if (cudaEventCreate(&g_prof.ev[c][e]) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    g_prof.created = true;
  }
  for (int e = 0; e < SS_NUM_PHASES; ++e) g_prof.ran[g_prof.used][e] = false;
  return true;
}

static int sm_count_of_current_device() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 148; }
  if (dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = 148;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

static int32_t check_desc(const ss_attn_desc_t* d) {
  if (!d || d->struct_size != sizeof(ss_attn_desc_t)) return SS_ERR_INVALID_ARG;
  if (d->flags & ~(SS_FLAG_VALIDATE | SS_FLAG_FORCE_GENERIC | SS_FLAG_NO_TCGEN05 | SS_FLAG_TILES_2CTA)) return SS_ERR_INVALID_ARG;
  if (d->num_q_heads < 1 || d->num_kv_heads < 1 || d->num_nodes < 0 || d->num_paths < 0 || d->total_q < 0 ||
      d->total_node_pages < 0 || d->num_pages < 0 || d->max_depth < 0 || d->max_decode_paths < 0 || d->max_sms < 0)
    return SS_ERR_INVALID_ARG;
  if (d->head_dim != kHeadDim || d->page_size != kPage) return SS_ERR_UNSUPPORTED;
  if (d->num_q_heads % d->num_kv_heads) return SS_ERR_UNSUPPORTED;
  if (d->num_q_heads / d->num_kv_heads > kTileRows) return SS_ERR_UNSUPPORTED;
  if (d->max_depth > SS_MAX_DEPTH) return SS_ERR_UNSUPPORTED;
  if (d->kv_token_stride != kHeadDim || d->kv_page_stride % 128 || d->kv_head_stride % 128 ||
      d->kv_page_stride <= 0 || d->kv_head_stride <= 0)
    return SS_ERR_UNSUPPORTED;
  if (!(d->sm_scale >= 0.f) || isinf(d->sm_scale)) return SS_ERR_INVALID_ARG;
  return SS_OK;
}

struct Layout {
  size_t total;
  Caps caps;
};

// Fills the workspace pointers of P (relative to `base`, which may be null for a pure size query).
static Layout carve(const ss_attn_desc_t* d, char* base, Params* P) {
  const int Hkv = d->num_kv_heads, G = d->num_q_heads / d->num_kv_heads;
  const int tpt = kTileRows / G;
  const int max_depth = d->max_depth > 0 ? d->max_depth : SS_MAX_DEPTH;
  const int64_t cap_dec = d->max_decode_paths > 0 ? (d->max_decode_paths < d->num_paths ? d->max_decode_paths : d->num_paths)
                                                  : d->num_paths;
  const int target = 2 * sm_count_of_current_device();   // (the size query and the call must see the same device)
  // Keys per leaf item.  (Finer items - 128 or 64 keys - were measured on the small configurations, where a warp of
  // the leaf kernel gets fewer than two items: the extra partials, counters and merges cost more than the better
  // balance gains, 0.50 -> 0.41 of the HBM rate at 64 keys; whole-leaf items of up to 512 keys: no gain either.)
  const int leaf_chunk = kLeafChunk;
  Caps caps;
  caps.dec = static_cast<int32_t>(cap_dec);
  const int64_t stacked = static_cast<int64_t>(Hkv) * (cap_dec * max_depth / tpt + d->num_nodes) + target + Hkv * kMaxRootSplits;
  const int64_t chain = static_cast<int64_t>(Hkv) * (d->total_q / tpt + d->num_paths);
  caps.tile_items = static_cast<int32_t>(stacked + chain);
  caps.leaf_items = static_cast<int32_t>(static_cast<int64_t>(Hkv) * (d->total_node_pages * kPage / leaf_chunk + cap_dec));
  caps.slots = cap_dec * (kMaxRootSplits + max_depth) + d->total_node_pages * kPage / leaf_chunk;

  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return base ? base + o : nullptr; };
  const size_t N = static_cast<size_t>(d->num_nodes) + 1, NP = static_cast<size_t>(d->num_paths) + 1;
  char* hdr = take(sizeof(PlanHeader));
  char* node_arrays[11];
  for (int i = 0; i < 11; ++i) node_arrays[i] = take(N * 4);
  char* path_arrays[6];
  for (int i = 0; i < 6; ++i) path_arrays[i] = take(NP * 4);
  char* dec_tok = take((static_cast<size_t>(cap_dec) + 1) * 4);
  char* dec_src = take((static_cast<size_t>(cap_dec) + 1) * 4);
  char* dec_slot = take((static_cast<size_t>(cap_dec) + 1) * 4);
  char* dec_chunks = take((static_cast<size_t>(cap_dec) + 1) * 4);
  char* leaf_arrive = take((static_cast<size_t>(cap_dec) * Hkv + 1) * 4);
  char* tiles = take(static_cast<size_t>(caps.tile_items) * sizeof(TileItem));
  char* leaves = take(static_cast<size_t>(caps.leaf_items) * sizeof(LeafItem));
  char* part_o = take(static_cast<size_t>(caps.slots) * d->num_q_heads * kHeadDim * 4);
  char* part_lse = take(static_cast<size_t>(caps.slots) * d->num_q_heads * 4);
  if (P) {
    P->hdr = reinterpret_cast<PlanHeader*>(hdr);
    int32_t** np[11] = {&P->node_start, &P->node_depth, &P->node_first, &P->node_last, &P->node_npaths, &P->node_ndec,
                        &P->node_own_slots, &P->node_level_off, &P->node_item_base, &P->node_splits, &P->node_split_len};
    for (int i = 0; i < 11; ++i) *np[i] = reinterpret_cast<int32_t*>(node_arrays[i]);
    int32_t** pp[6] = {&P->path_class, &P->path_kv_len, &P->path_dec_rank, &P->path_slot_base, &P->path_leaf_base,
                       &P->path_chain_base};
    for (int i = 0; i < 6; ++i) *pp[i] = reinterpret_cast<int32_t*>(path_arrays[i]);
    P->dec_tok = reinterpret_cast<int32_t*>(dec_tok);
    P->dec_src = reinterpret_cast<int32_t*>(dec_src);
    P->dec_slot_base = reinterpret_cast<int32_t*>(dec_slot);
    P->dec_leaf_chunks = reinterpret_cast<int32_t*>(dec_chunks);
    P->leaf_arrive = reinterpret_cast<int32_t*>(leaf_arrive);
    P->tile_items = reinterpret_cast<TileItem*>(tiles);
    P->leaf_items = reinterpret_cast<LeafItem*>(leaves);
    P->part_o = reinterpret_cast<float*>(part_o);
    P->part_lse = reinterpret_cast<float*>(part_lse);
    P->caps = caps;
    P->target_tiles = target;
    P->leaf_chunk = leaf_chunk;
  }
  Layout L;
  L.total = off;
  L.caps = caps;
  return L;
}

}  // namespace attn
}  // namespace ss

extern "C" int32_t ss_tree_attention_workspace_bytes(const ss_attn_desc_t* desc, size_t* out_bytes) {
  using namespace ss::attn;
  if (!out_bytes) return SS_ERR_INVALID_ARG;
  const int32_t rc = check_desc(desc);
  if (rc != SS_OK) return rc;
  *out_bytes = carve(desc, nullptr, nullptr).total;
  return SS_OK;
}

extern "C" int32_t ss_tree_attention(const ss_attn_desc_t* d, void* workspace, size_t workspace_bytes, void* stream) {
  using namespace ss;
  using namespace ss::attn;
  int32_t rc = check_desc(d);
  if (rc != SS_OK) return rc;
  if (!workspace || reinterpret_cast<uintptr_t>(workspace) % kAlign) return SS_ERR_INVALID_ARG;
  if (!d->k_pool || !d->v_pool || !d->node_parent || !d->node_kv_len || !d->node_page_offsets || !d->node_pages ||
      !d->path_leaf_node || !d->path_q_len || !d->q_offsets)
    return SS_ERR_INVALID_ARG;
  if (d->total_q > 0 && (!d->q || !d->out)) return SS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d->k_pool) % 256 || reinterpret_cast<uintptr_t>(d->v_pool) % 256 ||
      reinterpret_cast<uintptr_t>(d->q) % 16 || reinterpret_cast<uintptr_t>(d->out) % 32)
    return SS_ERR_UNSUPPORTED;
  if (d->total_q > 0x7fffffffLL / d->num_q_heads) return SS_ERR_UNSUPPORTED;   // row indices are int32
  if (d->total_node_pages > 0x7fffffffLL) return SS_ERR_UNSUPPORTED;           // so are indices into node_pages
  if (d->q_src_offsets && (d->q_src_rows < 0 || d->q_src_rows > 0x7fffffffLL / d->num_q_heads)) return SS_ERR_INVALID_ARG;

  Params P;
  memset(&P, 0, sizeof P);
  const Layout L = carve(d, static_cast<char*>(workspace), &P);
  if (workspace_bytes < L.total) return SS_ERR_WORKSPACE_TOO_SMALL;
  P.Hq = d->num_q_heads;
  P.Hkv = d->num_kv_heads;
  P.G = P.Hq / P.Hkv;
  P.tok_per_tile = kTileRows / P.G;
  P.scale = d->sm_scale > 0.f ? d->sm_scale : 1.0f / sqrtf(static_cast<float>(kHeadDim));
  P.scale_log2 = P.scale * 1.4426950408889634f;
  P.flags = d->flags;
  P.k_pool = static_cast<const __nv_bfloat16*>(d->k_pool);
  P.v_pool = static_cast<const __nv_bfloat16*>(d->v_pool);
  P.num_pages = d->num_pages;
  P.page_stride = d->kv_page_stride;
  P.head_stride = d->kv_head_stride;
  P.token_stride = d->kv_token_stride;
  P.num_nodes = d->num_nodes;
  P.node_parent = d->node_parent;
  P.node_kv_len = d->node_kv_len;
  P.node_page_offsets = d->node_page_offsets;
  P.node_pages = d->node_pages;
  P.total_node_pages = d->total_node_pages;
  P.num_paths = d->num_paths;
  P.num_paths_dev = d->num_paths_dev;
  P.path_leaf_node = d->path_leaf_node;
  P.path_q_len = d->path_q_len;
  P.q_offsets = d->q_offsets;
  P.q_src_offsets = d->q_src_offsets;
  P.q_src_rows = d->q_src_rows;
  P.total_q = d->total_q;
  P.q = static_cast<const __nv_bfloat16*>(d->q);
  P.out = static_cast<__nv_bfloat16*>(d->out);
  P.lse = d->lse;

  cudaStream_t st = as_stream(stream);
  int sms = sm_count_of_current_device();
  if (d->max_sms > 0 && d->max_sms < sms) sms = d->max_sms;
  const bool timed = prof_begin_call();
  const int call = g_prof.used;
  // phase boundaries: event e is recorded before phase e, event SS_NUM_PHASES after the last one
  auto mark = [&](int e) { if (timed) cudaEventRecord(g_prof.ev[call][e], st); };
  auto ran = [&](int e) { if (timed) g_prof.ran[call][e] = true; };
  const bool simple = (d->flags & SS_FLAG_NO_TCGEN05) != 0, generic_only = (d->flags & SS_FLAG_FORCE_GENERIC) != 0;
  const bool any = d->num_paths > 0 && d->total_q > 0;
  mark(SS_PHASE_PLAN);
  rc = launch_plan(P, st);
  ran(SS_PHASE_PLAN);
  mark(SS_PHASE_TILES);
  if (rc == SS_OK && any && !generic_only) {
    const bool two_cta = (d->flags & SS_FLAG_TILES_2CTA) != 0;
    rc = simple ? launch_tile_items_simple(P, st, sms)
                : (two_cta ? launch_tile_items_umma(P, st, sms) : launch_tile_items_umma_split(P, st, sms));
    ran(SS_PHASE_TILES);
  }
  // Decode leaves.  The streaming kernel also merges the per-level partials and computes the rows of GENERIC paths;
  // pools it cannot take (and the plain mode) go through the register-staged leaf kernel and a merge launch.
  const bool fused_finish = !simple && !generic_only && leaf_stream_supported(P);
  mark(SS_PHASE_LEAVES);
  if (rc == SS_OK && any && !generic_only) {
    rc = simple ? launch_leaf_items_simple(P, st, sms) : (fused_finish ? launch_leaf_stream(P, st, sms) : launch_leaf_items(P, st, sms));
    ran(SS_PHASE_LEAVES);
  }
  mark(SS_PHASE_GENERIC);
  if (rc == SS_OK && any && generic_only) {
    rc = launch_generic(P, st, sms);
    ran(SS_PHASE_GENERIC);
  }
  mark(SS_PHASE_MERGE);
  if (rc == SS_OK && any && !generic_only && !fused_finish) {
    rc = launch_merge(P, st, sms);                    // (rows of GENERIC paths, then the merge)
    ran(SS_PHASE_MERGE);
  }
  mark(SS_NUM_PHASES);
  if (timed) ++g_prof.used;
  return rc;
}

extern "C" int32_t ss_profile_enable(int32_t on) {
  ss::attn::g_prof.on = on != 0;
  return SS_OK;
}

extern "C" int32_t ss_profile_read(float* phase_ms, int64_t* phase_calls) {
  using namespace ss::attn;
  float ms[SS_NUM_PHASES] = {0};
  int64_t calls[SS_NUM_PHASES] = {0};
  int32_t rc = SS_OK;
  for (int c = 0; c < g_prof.used; ++c) {
    if (cudaEventSynchronize(g_prof.ev[c][SS_NUM_PHASES]) != cudaSuccess) { (void)cudaGetLastError(); rc = SS_ERR_CUDA; break; }
    for (int e = 0; e < SS_NUM_PHASES; ++e) {
      if (!g_prof.ran[c][e]) continue;
      float t = 0.f;
      if (cudaEventElapsedTime(&t, g_prof.ev[c][e], g_prof.ev[c][e + 1]) != cudaSuccess) { (void)cudaGetLastError(); rc = SS_ERR_CUDA; continue; }
      ms[e] += t;
      calls[e] += 1;
    }
  }
  g_prof.used = 0;
  for (int e = 0; e < SS_NUM_PHASES; ++e) {
    if (phase_ms) phase_ms[e] = ms[e];
    if (phase_calls) phase_calls[e] = calls[e];
  }
  return rc;
}
