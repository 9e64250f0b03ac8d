// One query row per warp, keys visited one at a time with an online softmax, all in fp32: lane l owns dims 4l..4l+3
// of q and of the output accumulator.  Shared by the plain kernels (attn_simple.cu) and by the exact second pass of
// the tensor-core tile kernel (a tile item whose scores left the range of its lagged reference maximum).
#pragma once
#include "attn_plan.cuh"

namespace ss {
namespace attn {

struct RowState {
  float q[4];
  float acc[4];
  float m, l;
};

__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&u.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&u.y);
  v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}

__device__ __forceinline__ void row_init(RowState& r, const __nv_bfloat16* qrow, int lane) {
  load4(qrow + 4 * lane, r.q);
  r.acc[0] = r.acc[1] = r.acc[2] = r.acc[3] = 0.f;
  r.m = -INFINITY;
  r.l = 0.f;
}

// Visit keys [t0, t1) of one node (t relative to the node).
__device__ __forceinline__ void row_visit_node(RowState& r, const Params& P, int node, int g, int t0, int t1, int lane) {
  if (t1 <= t0) return;
  const int64_t pg0 = P.node_page_offsets[node];
  for (int t = t0; t < t1; ++t) {
    const int64_t page = P.node_pages[pg0 + t / kPage];
    const int64_t off = page * P.page_stride + static_cast<int64_t>(g) * P.head_stride +
                        static_cast<int64_t>(t % kPage) * P.token_stride + 4 * lane;
    float k[4], v[4];
    load4(P.k_pool + off, k);
    float s = r.q[0] * k[0] + r.q[1] * k[1] + r.q[2] * k[2] + r.q[3] * k[3];
    s = warp_sum(s) * P.scale;
    load4(P.v_pool + off, v);
    const float m_new = fmaxf(r.m, s);
    const float corr = __expf(r.m - m_new);          // exp(-inf) = 0 on the first key
    const float p = __expf(s - m_new);
    r.l = r.l * corr + p;
#pragma unroll
    for (int i = 0; i < 4; ++i) r.acc[i] = r.acc[i] * corr + p * v[i];
    r.m = m_new;
  }
}

__device__ __forceinline__ void row_store_final(const RowState& r, const Params& P, int64_t q_row, int h, int lane) {
  const float inv = r.l > 0.f ? 1.f / r.l : 0.f;
  __nv_bfloat16* o = P.out + (q_row * P.Hq + h) * kHeadDim + 4 * lane;
  __nv_bfloat162 a = __floats2bfloat162_rn(r.acc[0] * inv, r.acc[1] * inv);
  __nv_bfloat162 b = __floats2bfloat162_rn(r.acc[2] * inv, r.acc[3] * inv);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(o) = u;
  if (P.lse && lane == 0) P.lse[q_row * P.Hq + h] = r.l > 0.f ? r.m + __logf(r.l) : -INFINITY;
}

__device__ __forceinline__ void row_store_partial(const RowState& r, const Params& P, int64_t slot, int h, int lane) {
  const float inv = r.l > 0.f ? 1.f / r.l : 0.f;
  float4 o = make_float4(r.acc[0] * inv, r.acc[1] * inv, r.acc[2] * inv, r.acc[3] * inv);
  *reinterpret_cast<float4*>(P.part_o + (slot * P.Hq + h) * kHeadDim + 4 * lane) = o;
  if (lane == 0) P.part_lse[slot * P.Hq + h] = r.l > 0.f ? r.m + __logf(r.l) : -INFINITY;
}

// Keys [v0, v1) of the virtual sequence root -> `leaf` (chain nodes concatenated).
__device__ inline void row_visit_chain(RowState& r, const Params& P, int leaf, int g, int v0, int v1, int lane) {
  int chain[SS_MAX_DEPTH];
  int d = 0;
  for (int a = leaf; a >= 0 && d < SS_MAX_DEPTH; a = P.node_parent[a]) chain[d++] = a;
  for (int c = d - 1; c >= 0; --c) {
    const int n = chain[c];
    const int start = P.node_start[n], len = P.node_kv_len[n];
    const int t0 = max(v0 - start, 0), t1 = min(v1 - start, len);
    row_visit_node(r, P, n, g, t0, t1, lane);
  }
}

// One tile item, exactly: rows `warp_index`, `warp_index + n_warps`, ... of the item, one warp each (whole warps).
__device__ __forceinline__ void tile_item_rows_exact(const Params& P, const TileItem& it, int warp_index, int n_warps, int lane) {
  const int kind = it.kind_g >> 16, g = it.kind_g & 0xffff;
  const int rows = it.n_tok * P.G;
  for (int rrow = warp_index; rrow < rows; rrow += n_warps) {
    const int i = rrow / P.G, h = g * P.G + rrow % P.G;
    const int dec = it.tok0 + i;                       // stacked: index into dec_tok
    const int64_t q_row = (kind == kItemChain) ? static_cast<int64_t>(it.tok0 + i) : P.dec_tok[dec];
    const int64_t q_src = (kind == kItemChain) ? static_cast<int64_t>(it.src0 + i) : P.dec_src[dec];
    const int visible = (kind == kItemChain) ? it.limit0 + i : it.limit0;
    const int v1 = min(it.kv_end, visible);
    RowState r;
    row_init(r, P.q + (q_src * P.Hq + h) * kHeadDim, lane);
    if (kind == kItemChain) {
      row_visit_chain(r, P, it.node, g, it.kv_begin, v1, lane);
      row_store_final(r, P, q_row, h, lane);
    } else {
      row_visit_node(r, P, it.node, g, it.kv_begin, v1, lane);
      row_store_partial(r, P, static_cast<int64_t>(P.dec_slot_base[dec]) + it.slot_off, h, lane);
    }
  }
}

}  // namespace attn
}  // namespace ss
