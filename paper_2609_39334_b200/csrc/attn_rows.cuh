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
    int64_t page = P.node_pages[pg0 + t / kPage];
    SS_CHECK_OR(page >= 0 && page < P.num_pages, &P.hdr->status, page = 0);
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

// Log-sum-exp merge of the per-level partial results of decode token `d`, q head `h` (one whole warp):
// out = sum_s exp(lse_s - LSE) o_s,  LSE = log sum_s exp(lse_s); a token without partials (no keys) gives 0 / -inf.
// The partials are read from L2 (ld.global.cg): inside the leaf kernel they may have been written by other SMs
// moments ago.
__device__ __forceinline__ void merge_row(const Params& P, int d, int h, int lane) {
  const int s0 = P.dec_slot_base[d], s1 = P.dec_slot_base[d + 1];
  SS_CHECK_OR(s0 >= 0 && s0 <= s1 && s1 <= P.caps.slots && P.dec_tok[d] >= 0 && P.dec_tok[d] < P.total_q, &P.hdr->status,
              return);
  float m = -INFINITY;
  for (int s = s0 + lane; s < s1; s += 32) m = fmaxf(m, __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h));
  m = warp_max(m);
  RowState r;
  r.acc[0] = r.acc[1] = r.acc[2] = r.acc[3] = 0.f;
  r.l = 0.f;
  r.m = m;
  if (m > -INFINITY) {
    for (int s = s0; s < s1; ++s) {
      const float ls = __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h);
      if (ls == -INFINITY) continue;
      const float wgt = __expf(ls - m);
      const float4 o = __ldcg(reinterpret_cast<const float4*>(P.part_o + (static_cast<int64_t>(s) * P.Hq + h) * kHeadDim + 4 * lane));
      r.l += wgt;
      r.acc[0] += wgt * o.x; r.acc[1] += wgt * o.y; r.acc[2] += wgt * o.z; r.acc[3] += wgt * o.w;
    }
  }
  row_store_final(r, P, P.dec_tok[d], h, lane);
}

// The same merge for the (up to 8) q heads [h0, h0 + n_rows) of decode token `d` at once (one whole warp).  The rows
// are independent, so their loads are issued together: merging them one after another costs two memory round trips
// per row, which is what a leaf item's last warp would otherwise wait for.
__device__ __forceinline__ void merge_rows8(const Params& P, int d, int h0, int n_rows, int lane) {
  int s0 = P.dec_slot_base[d], s1 = P.dec_slot_base[d + 1];
  SS_CHECK_OR(s0 >= 0 && s0 <= s1 && s1 <= P.caps.slots && P.dec_tok[d] >= 0 && P.dec_tok[d] < P.total_q, &P.hdr->status,
              return);
  float m[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    m[r] = -INFINITY;
    if (r < n_rows)
      for (int s = s0 + lane; s < s1; s += 32) m[r] = fmaxf(m[r], __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h0 + r));
  }
#pragma unroll
  for (int r = 0; r < 8; ++r) m[r] = warp_max(m[r]);
  float acc[8][4], l[8];
#pragma unroll
  for (int r = 0; r < 8; ++r) { acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f; l[r] = 0.f; }
  for (int s = s0; s < s1; ++s) {
    float ls[8];
    float4 o[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      ls[r] = -INFINITY;
      o[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < n_rows) {
        ls[r] = __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h0 + r);
        o[r] = __ldcg(reinterpret_cast<const float4*>(P.part_o + (static_cast<int64_t>(s) * P.Hq + h0 + r) * kHeadDim + 4 * lane));
      }
    }
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      const float wgt = ls[r] == -INFINITY ? 0.f : __expf(ls[r] - m[r]);   // (m = -inf only if every ls is)
      l[r] += wgt;
      acc[r][0] += wgt * o[r].x; acc[r][1] += wgt * o[r].y; acc[r][2] += wgt * o[r].z; acc[r][3] += wgt * o[r].w;
    }
  }
  const int64_t q_row = P.dec_tok[d];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    if (r >= n_rows) continue;
    RowState rs;
    rs.acc[0] = acc[r][0]; rs.acc[1] = acc[r][1]; rs.acc[2] = acc[r][2]; rs.acc[3] = acc[r][3];
    rs.l = l[r];
    rs.m = m[r];
    row_store_final(rs, P, q_row, h0 + r, lane);
  }
}

// Rows of GENERIC paths: warp `w` of `warps` takes rows w, w + warps, ... of all (query token, q head) rows.
__device__ inline void generic_rows(const Params& P, int64_t w, int64_t warps, int lane) {
  const int live = P.hdr->live_paths;
  if (live <= 0) return;
  const int64_t total_rows = P.q_offsets[live] * P.Hq;
  for (; w < total_rows; w += warps) {
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

}  // namespace attn
}  // namespace ss
