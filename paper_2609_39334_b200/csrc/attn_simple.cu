// Simple attention kernels of ss_tree_attention:
//   generic_kernel        one warp per (query token, q head) walking the path's whole chain; takes every
//                         shape (class GENERIC, or everything under SS_FLAG_FORCE_GENERIC)
//   tile_items_simple     executes the planner's tile items one warp per stacked row (SS_FLAG_NO_TCGEN05):
//                         the same plan as the tensor-core kernel, without tensor cores
//   leaf_items_simple     executes leaf items one warp per (item, q head of the group)
//   merge_kernel          rows of GENERIC paths, then the log-sum-exp merge of the per-level partial results of
//                         decode tokens (the fallback when the streaming leaf kernel, which merges itself, is not used)
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
  generic_rows(P, (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5, warps, lane);
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

// Generic rows (if any) and the log-sum-exp merge of every decode token, in one launch.
__global__ void merge_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;
  const int lane = threadIdx.x & 31;
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  const int64_t w0 = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
  if (P.hdr->n_generic_rows > 0) generic_rows(P, w0, warps, lane);
  const int64_t total = static_cast<int64_t>(P.hdr->n_dec) * P.Hq;
  for (int64_t w = w0; w < total; w += warps) merge_row(P, static_cast<int>(w / P.Hq), static_cast<int>(w % P.Hq), lane);
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
