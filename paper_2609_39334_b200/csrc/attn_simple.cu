// Simple attention kernels of ss_tree_attention:
//   generic_kernel        one warp per (query token, q head) walking the path's whole chain; takes every
//                         shape (class GENERIC, or everything under SS_FLAG_FORCE_GENERIC)
//   tile_items_simple     executes the planner's tile items one warp per stacked row (SS_FLAG_NO_TCGEN05):
//                         the same plan as the tensor-core kernel, without tensor cores
//   leaf_items_simple     executes leaf items one warp per (item, q head of the group)
//   merge_kernel          log-sum-exp merge of the per-level partial results of decode tokens
// A warp holds one query row: lane l owns dims 4l..4l+3 of q and of the output accumulator; keys are visited one
// at a time with an online softmax (running max m, running sum l), all in fp32.
#include "attn_rows.cuh"

namespace ss {
namespace attn {

// ---------------------------------------------------------------------------------------------------------
__global__ void generic_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK || P.hdr->n_generic_rows == 0) return;
  const int lane = threadIdx.x & 31;
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  const int live = P.hdr->live_paths;
  if (live <= 0) return;
  const int64_t total_rows = P.q_offsets[live] * P.Hq;
  for (int64_t w = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; w < total_rows; w += warps) {
    const int64_t q_row = w / P.Hq;
    const int h = static_cast<int>(w % P.Hq);
    int lo = 0, hi = live;                    // path with q_offsets[p] <= q_row < q_offsets[p+1]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (P.q_offsets[mid] <= q_row) lo = mid; else hi = mid;
    }
    const int p = lo;
    if (P.path_class[p] != kClassGeneric) continue;
    const int T = P.path_q_len[p];
    const int t = static_cast<int>(q_row - P.q_offsets[p]);
    const int visible = P.path_kv_len[p] - T + t + 1;
    RowState r;
    const int64_t q_src = P.q_src_offsets ? P.q_src_offsets[p] + t : q_row;
    row_init(r, P.q + (q_src * P.Hq + h) * kHeadDim, lane);
    if (visible > 0) row_visit_chain(r, P, P.path_leaf_node[p], h / P.G, 0, visible, lane);
    row_store_final(r, P, q_row, h, lane);
  }
}

__global__ void tile_items_simple(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int n_items = P.hdr->n_tile_items;
  for (int e = blockIdx.x; e < n_items; e += gridDim.x) tile_item_rows_exact(P, P.tile_items[e], warp, nw, lane);
}

__global__ void leaf_items_simple(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;
  const int lane = threadIdx.x & 31;
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  const int64_t total = static_cast<int64_t>(P.hdr->n_leaf_items) * P.G;
  for (int64_t w = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; w < total; w += warps) {
    const LeafItem it = P.leaf_items[w / P.G];
    const int h = it.g * P.G + static_cast<int>(w % P.G);
    RowState r;
    row_init(r, P.q + (static_cast<int64_t>(it.q_src) * P.Hq + h) * kHeadDim, lane);
    row_visit_node(r, P, it.node, it.g, it.kv_begin, it.kv_end, lane);
    row_store_partial(r, P, it.slot, h, lane);
  }
}

// out = sum_s exp(lse_s - LSE) o_s,  LSE = log sum_s exp(lse_s); a token without partials (no keys) gives 0 / -inf.
__global__ void merge_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;
  const int lane = threadIdx.x & 31;
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  const int64_t total = static_cast<int64_t>(P.hdr->n_dec) * P.Hq;
  for (int64_t w = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; w < total; w += warps) {
    const int d = static_cast<int>(w / P.Hq), h = static_cast<int>(w % P.Hq);
    const int s0 = P.dec_slot_base[d], s1 = P.dec_slot_base[d + 1];
    float m = -INFINITY;
    for (int s = s0 + lane; s < s1; s += 32) m = fmaxf(m, P.part_lse[static_cast<int64_t>(s) * P.Hq + h]);
    m = warp_max(m);
    RowState r;
    r.acc[0] = r.acc[1] = r.acc[2] = r.acc[3] = 0.f;
    r.l = 0.f;
    r.m = m;
    if (m > -INFINITY) {
      for (int s = s0; s < s1; ++s) {
        const float ls = P.part_lse[static_cast<int64_t>(s) * P.Hq + h];
        if (ls == -INFINITY) continue;
        const float wgt = __expf(ls - m);
        const float4 o = *reinterpret_cast<const float4*>(P.part_o + (static_cast<int64_t>(s) * P.Hq + h) * kHeadDim + 4 * lane);
        r.l += wgt;
        r.acc[0] += wgt * o.x; r.acc[1] += wgt * o.y; r.acc[2] += wgt * o.z; r.acc[3] += wgt * o.w;
      }
    }
    row_store_final(r, P, P.dec_tok[d], h, lane);
  }
}

int32_t launch_generic(const Params& P, cudaStream_t st, int sm_count) {
  SS_LAUNCH(generic_kernel, sm_count * 8, 256, 0, st, P);
  return SS_OK;
}
int32_t launch_tile_items_simple(const Params& P, cudaStream_t st, int sm_count) {
  SS_LAUNCH(tile_items_simple, sm_count * 4, 256, 0, st, P);
  return SS_OK;
}
int32_t launch_leaf_items_simple(const Params& P, cudaStream_t st, int sm_count) {
  SS_LAUNCH(leaf_items_simple, sm_count * 8, 256, 0, st, P);
  return SS_OK;
}
int32_t launch_merge(const Params& P, cudaStream_t st, int sm_count) {
  SS_LAUNCH(merge_kernel, sm_count * 8, 256, 0, st, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
