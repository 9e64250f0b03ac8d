// Decode-leaf attention (bandwidth-bound): one warp per leaf item = (decode token, kv head, chunk of <= 256 keys of
// the path's private leaf).  The G query rows of the GQA group (padded to 16) go through warp-level
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate) so that the per-key arithmetic stays far below the HBM time;
// K and V come straight from global memory into registers with 128-bit loads - no shared memory, no barriers:
//
//   * QK^T: the dot product over the 128 dims does not care about the order of the dims, so every thread loads
//     16 contiguous bytes (8 dims) of one key row and uses them as the k-slots the MMA fragment layout assigns to
//     that thread; the query fragments are loaded once with the same dim permutation.
//   * PV: every thread loads 16 contiguous bytes (8 output dims) of the four key rows whose k-slots it owns and
//     pairs rows with byte-permutes; the 8 dims feed 8 MMAs, i.e. the output dims are permuted the same way and
//     un-permuted when the partial result is written.
//
// Online softmax in the exp2 domain with quad shuffles (a query row lives in the 4 lanes of a quad).  Each item
// writes a normalised fp32 partial (o, lse) that the merge kernel combines with the shared-node partials.
#include "attn_plan.cuh"

namespace ss {
namespace attn {

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint4 ldg128(const __nv_bfloat16* p) {
  return __ldg(reinterpret_cast<const uint4*>(p));
}

constexpr int kLeafWarps = 4;

// TWO: the GQA group has more than 8 rows (rows gid and gid+8 of the MMA tile are both live).
template <bool TWO>
__global__ void __launch_bounds__(kLeafWarps * 32) leaf_items_kernel(const Params P) {
  ss::grid_dependency_enter();
  if (P.hdr->status != SS_OK) return;
  const int lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int n_items = P.hdr->n_leaf_items;
  const int G = P.G;
  const float c = P.scale_log2;

  for (;;) {
    int e = 0;
    if (lane == 0) e = atomicAdd(&P.hdr->leaf_counter, 1);
    e = __shfl_sync(0xffffffffu, e, 0);
    if (e >= n_items) break;
    const LeafItem it = P.leaf_items[e];
    const int n_keys = it.kv_end - it.kv_begin;
    const int n_pages = (n_keys + kPage - 1) / kPage;                      // <= 16
    const int64_t pg0 = P.node_page_offsets[it.node] + it.kv_begin / kPage;
    int my_page = lane < n_pages ? P.node_pages[pg0 + lane] : 0;
    SS_CHECK_OR(my_page >= 0 && my_page < P.num_pages, &P.hdr->status, my_page = 0);
    bool slot_ok = true;
    (void)slot_ok;
    SS_CHECK_OR(it.slot >= 0 && it.slot < P.caps.slots, &P.hdr->status, slot_ok = false);

    // ---- query fragments (dim-permuted, see above) --------------------------------------------------------
    uint4 qa[4], qb[4];
    {
      const __nv_bfloat16* q0 = P.q + (static_cast<int64_t>(it.q_src) * P.Hq + it.g * G) * kHeadDim;
#pragma unroll
      for (int k2 = 0; k2 < 4; ++k2) {
        qa[k2] = gid < G ? ldg128(q0 + gid * kHeadDim + 32 * k2 + 8 * tig) : make_uint4(0, 0, 0, 0);
        if (TWO) qb[k2] = gid + 8 < G ? ldg128(q0 + (gid + 8) * kHeadDim + 32 * k2 + 8 * tig) : make_uint4(0, 0, 0, 0);
        else qb[k2] = make_uint4(0, 0, 0, 0);
      }
    }
    float o[2][8][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int j = 0; j < 8; ++j) o[a][j][0] = o[a][j][1] = o[a][j][2] = o[a][j][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;              // rows gid and gid+8

    uint4 kreg[2][4];
    auto load_k = [&](int pg) {
      const int page = __shfl_sync(0xffffffffu, my_page, pg);
      const __nv_bfloat16* kb = P.k_pool + static_cast<int64_t>(page) * P.page_stride + static_cast<int64_t>(it.g) * P.head_stride;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2) kreg[nt][k2] = ldg128(kb + (gid + 8 * nt) * kHeadDim + 32 * k2 + 8 * tig);
    };
    load_k(0);

    for (int pg = 0; pg < n_pages; ++pg) {
      const int valid = min(kPage, n_keys - pg * kPage);                   // keys of this page that exist
      const int page = __shfl_sync(0xffffffffu, my_page, pg);
      const __nv_bfloat16* vb = P.v_pool + static_cast<int64_t>(page) * P.page_stride + static_cast<int64_t>(it.g) * P.head_stride;
      // V rows of the four keys whose k-slots this thread owns, two 8-dim chunks each
      uint4 vreg[2][4];
#pragma unroll
      for (int hq = 0; hq < 2; ++hq)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int tv = 2 * tig + (r & 1) + 8 * (r >> 1);
          vreg[hq][r] = ldg128(vb + tv * kHeadDim + (gid + 8 * hq) * 8);
        }
      // ---- S = Q K^T ------------------------------------------------------------------------------------------
      float s[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2) {
          mma_bf16_16816(s[nt], qa[k2].x, qb[k2].x, qa[k2].y, qb[k2].y, kreg[nt][k2].x, kreg[nt][k2].y);
          mma_bf16_16816(s[nt], qa[k2].z, qb[k2].z, qa[k2].w, qb[k2].w, kreg[nt][k2].z, kreg[nt][k2].w);
        }
      }
      if (pg + 1 < n_pages) load_k(pg + 1);                                // prefetch while the softmax runs
      // ---- mask the tail of the last page (slots past the length hold undefined data) --------------------------
      if (valid < kPage) {
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
          for (int x = 0; x < 2; ++x)
            if (8 * nt + 2 * tig + x >= valid) { s[nt][x] = -INFINITY; s[nt][2 + x] = -INFINITY; }
#pragma unroll
        for (int hq = 0; hq < 2; ++hq)
#pragma unroll
          for (int r = 0; r < 4; ++r)
            if (2 * tig + (r & 1) + 8 * (r >> 1) >= valid) vreg[hq][r] = make_uint4(0, 0, 0, 0);
      }
      // ---- online softmax (row gid in s[.][0..1], row gid+8 in s[.][2..3]) ------------------------------------
      float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
      float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      if (TWO) {
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      }
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float ms0 = mn0 == -INFINITY ? 0.f : mn0 * c, ms1 = mn1 == -INFINITY ? 0.f : mn1 * c;
      const float corr0 = exp2f(m0 * c - ms0), corr1 = TWO ? exp2f(m1 * c - ms1) : 1.f;   // exp2(-inf) = 0
      m0 = mn0;
      m1 = mn1;
      float p[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        p[nt][0] = exp2f(s[nt][0] * c - ms0);
        p[nt][1] = exp2f(s[nt][1] * c - ms0);
        p[nt][2] = TWO ? exp2f(s[nt][2] * c - ms1) : 0.f;
        p[nt][3] = TWO ? exp2f(s[nt][3] * c - ms1) : 0.f;
      }
      float sum0 = p[0][0] + p[0][1] + p[1][0] + p[1][1];
      float sum1 = p[0][2] + p[0][3] + p[1][2] + p[1][3];
      l0 = l0 * corr0 + sum0;                                              // per-thread partial sums; quad-reduced at the end
      l1 = l1 * corr1 + sum1;
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          o[a][j][0] *= corr0; o[a][j][1] *= corr0;
          if (TWO) { o[a][j][2] *= corr1; o[a][j][3] *= corr1; }
        }
      // ---- O += P V ------------------------------------------------------------------------------------------------
      const uint32_t pa0 = pack_bf16(p[0][0], p[0][1]), pa1 = pack_bf16(p[0][2], p[0][3]);
      const uint32_t pa2 = pack_bf16(p[1][0], p[1][1]), pa3 = pack_bf16(p[1][2], p[1][3]);
#pragma unroll
      for (int hq = 0; hq < 2; ++hq) {
        const uint32_t* r0 = reinterpret_cast<const uint32_t*>(&vreg[hq][0]);
        const uint32_t* r1 = reinterpret_cast<const uint32_t*>(&vreg[hq][1]);
        const uint32_t* r2 = reinterpret_cast<const uint32_t*>(&vreg[hq][2]);
        const uint32_t* r3 = reinterpret_cast<const uint32_t*>(&vreg[hq][3]);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
          const uint32_t b0 = __byte_perm(r0[j >> 1], r1[j >> 1], sel);
          const uint32_t b1 = __byte_perm(r2[j >> 1], r3[j >> 1], sel);
          mma_bf16_16816(o[hq][j], pa0, pa1, pa2, pa3, b0, b1);
        }
      }
    }
    // ---- write the normalised partial ----------------------------------------------------------------------------
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    if (TWO) {
      l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    }
#pragma unroll
    for (int rg = 0; rg < (TWO ? 2 : 1); ++rg) {
      const int row = gid + 8 * rg;
      if (row >= G) continue;
#ifdef SS_CHECKED
      if (!slot_ok) continue;
#endif
      const float l = rg ? l1 : l0, m = rg ? m1 : m0;
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const int h = it.g * G + row;
      float* dst = P.part_o + (static_cast<int64_t>(it.slot) * P.Hq + h) * kHeadDim;
#pragma unroll
      for (int hq = 0; hq < 2; ++hq)
#pragma unroll
        for (int x = 0; x < 2; ++x) {                                       // x: MMA column 2*tig + x
          const int chunk = 2 * tig + x + 8 * hq;                           // dims chunk*8 .. chunk*8+7
          float4 lo = make_float4(o[hq][0][2 * rg + x] * inv, o[hq][1][2 * rg + x] * inv, o[hq][2][2 * rg + x] * inv,
                                  o[hq][3][2 * rg + x] * inv);
          float4 hi = make_float4(o[hq][4][2 * rg + x] * inv, o[hq][5][2 * rg + x] * inv, o[hq][6][2 * rg + x] * inv,
                                  o[hq][7][2 * rg + x] * inv);
          *reinterpret_cast<float4*>(dst + chunk * 8) = lo;
          *reinterpret_cast<float4*>(dst + chunk * 8 + 4) = hi;
        }
      if (tig == 0) P.part_lse[static_cast<int64_t>(it.slot) * P.Hq + h] = l > 0.f ? m * P.scale + __logf(l) : -INFINITY;
    }
  }
}

int32_t launch_leaf_items(const Params& P, cudaStream_t st, int sm_count) {
  const int blocks = sm_count * 8;
  if (P.G > 8) SS_LAUNCH(leaf_items_kernel<true>, blocks, kLeafWarps * 32, 0, st, P);
  else SS_LAUNCH(leaf_items_kernel<false>, blocks, kLeafWarps * 32, 0, st, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
