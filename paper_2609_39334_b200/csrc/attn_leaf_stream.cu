// Decode-leaf attention, streaming version (the default): bandwidth-bound, so what counts is bytes in flight.
// Every warp is a pipeline of its own: an elected lane streams the (page, kv head) blocks of K and V of the warp's
// leaf items through a private ring of shared memory with bulk-tensor copies (2 pages = 16 KB in flight per warp,
// 12 warps: ~190 KB per SM, three times what a register-staged loop can hold; groups of 9-16 query heads: 8 warps x
// 3 pages), and the warp consumes them with ldmatrix + mma.sync.m16n8k16 in transposed form (the 16 keys of a page
// are the M dimension, the query rows of the GQA group the N dimension; fp32 online softmax in the exp2 domain with
// shuffles).  The copies use the same tensor map as the tile kernel (each block lands as 128-byte-swizzled 8-row
// atoms), so the ldmatrix reads are free of bank conflicts.  Items are taken from a global counter; the NEXT item's
// descriptor, page ids and query rows are fetched while the current item is computed and its pages are requested as
// soon as ring stages free up, so the stream does not stop at item boundaries.
//
// The kernel also finishes the decode tokens: an item writes its normalised fp32 partial (o, lse), counts itself in
// leaf_arrive[token][kv head], and the warp that brings the count to the token's number of leaf chunks merges ALL
// partials of that (token, kv head) - the shared-node partials come from the tile kernel, for whose completion a
// warp waits before its first read of them - and writes the final bf16 rows.  Tokens without a private leaf, and rows of GENERIC
// paths, are swept after the items.  No separate merge launch.
#include "attn_plan.cuh"
#include "attn_rows.cuh"
#include "umma.cuh"

namespace ss {
namespace attn {
namespace leafs {

using namespace umma;

constexpr int kBlockBytes = 4096;          // one (page, kv head) block of K or of V: 16 rows x 256 B
constexpr int kStageBytes = 2 * kBlockBytes;
constexpr float kLazyLog2 = 8.0f;          // the running maximum of a row moves only when exceeded by 2^8

// NT: 8-row groups of query rows (1: GQA group <= 8, 2: <= 16).  WARPS x STAGES pages of 8 KB are in flight per SM.
template <int NT, int WARPS, int STAGES>
struct Cfg {
  static constexpr int kWarps = WARPS;
  static constexpr int kStages = STAGES;
  static constexpr int kRingBytes = STAGES * kStageBytes;
  static constexpr int kSmem = WARPS * kRingBytes + 1024;      // + slack for the 1024-byte alignment
};

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
// Transposes an 8 x 8 matrix of 16-bit elements held one row per quad-group (thread (gid, tig): row gid, columns
// 2 tig, 2 tig + 1).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct Item {            // one leaf item as a warp holds it (all lanes the same, except my_page)
  int valid;             // 0: the item list is exhausted
  int g, n_keys, slot, dec, n_pages;
  int chunks;            // leaf items of the token's leaf (per kv head)
  int my_page;           // lane l: physical page of the item's page l
};

// The products are taken transposed, so that the 16 keys of a page are the M dimension of one MMA and the (<= 8 NT)
// query rows of the GQA group its N dimension:
//   S^T[key][q] = K[key][dim] Q^T[dim][q]      A = K rows (ldmatrix), B = the query rows (registers, loaded per item)
//   O^T[dim][q] += V^T[dim][key] P^T[key][q]   A = V rows (ldmatrix.trans), B = P^T: the accumulator of S^T holds P one
//                                              key per quad-group, movmatrix turns it into the B fragment
// 8 + 8 MMAs per page and kv head for a group of up to 8 rows (the untransposed form needs 16 + 16 and twice the
// accumulator registers, half of them for padding rows).  A thread holds two query columns (2 tig, 2 tig + 1) per
// 8-row group: the running maxima and sums are per column, reduced over the 8 quad-groups by shuffles.
template <int NT, int WARPS, int STAGES>
__global__ void __launch_bounds__(WARPS * 32, 1)
leaf_stream_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const __grid_constant__ Params P) {
  // This kernel follows the tile kernel but its items need nothing from it: it starts as soon as SMs are free (the
  // tile kernel has waited for the planner before releasing it) and waits for the tile kernel only where it first
  // reads the shared-node partials - and in every thread before the kernel ends.
  ss::grid_dependency_release();
  using C = Cfg<NT, WARPS, STAGES>;
  constexpr int kStages = STAGES;
  SS_STAMP_BEGIN(P.hdr, 4);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t full_bar[WARPS][STAGES];
  __shared__ int abort_flag_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = lane >> 2, tig = lane & 3;
  volatile int* abort_flag = &abort_flag_s;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint8_t* ring_ptr = smem + warp * C::kRingBytes;
  const uint32_t ring = smem_u32(ring_ptr);
  if (tid == 0) {
    abort_flag_s = 0;
    prefetch_tensormap(&tmap_k);
    prefetch_tensormap(&tmap_v);
  }
  if (lane == 0)
    for (int s = 0; s < kStages; ++s) mbar_init(&full_bar[warp][s], 1);
  fence_barrier_init();
  __syncthreads();

  // (what the planner wrote is read from L2 until the dependency wait: this kernel's blocks start while the tile
  //  kernel is still running, on SMs whose L1 may hold lines from before the planner ran)
  const bool plan_ok = __ldcg(&P.hdr->status) == SS_OK;
  const int n_items = plan_ok ? __ldcg(&P.hdr->n_leaf_items) : 0;
  const int G = P.G;
  const float c = P.scale_log2;
  const float lazy_raw = kLazyLog2 / c;

  // ---- item fetch, in three steps so that its dependent loads can be spread over the page loop --------------------
  int f_e = 0;
  LeafItem f_it;
  uint32_t nq[NT][8][2];                                         // query fragments of the item being fetched
  bool first_claim = true;
  auto fetch_claim = [&]() {                                     // step 1: claim an item index
    // (a warp's first item is its own index in the grid - one trip to memory less before its first page - and the
    //  counter hands out the items after those)
    const int n_warps_grid = static_cast<int>(gridDim.x) * WARPS;
    if (first_claim) {
      f_e = static_cast<int>(blockIdx.x) * WARPS + warp;
      first_claim = false;
      return;
    }
    int e = 0;
    if (lane == 0) e = atomicAdd(&P.hdr->leaf_counter, 1) + n_warps_grid;
    f_e = __shfl_sync(0xffffffffu, e, 0);
  };
  auto fetch_desc = [&]() {                                      // step 2: its descriptor
    if (f_e < n_items) {
      const uint4* src = reinterpret_cast<const uint4*>(P.leaf_items + f_e);
      const uint4 lo = __ldcg(src), hi = __ldcg(src + 1);
      *reinterpret_cast<uint4*>(&f_it) = lo;
      *(reinterpret_cast<uint4*>(&f_it) + 1) = hi;
    }
  };
  auto fetch_finish = [&](Item& it) {                            // step 3: page ids, query rows
    it.valid = f_e < n_items ? 1 : 0;
    if (!it.valid) return;
    it.g = f_it.g; it.n_keys = f_it.kv_end - f_it.kv_begin; it.slot = f_it.slot; it.dec = f_it.dec;
    it.n_pages = (it.n_keys + kPage - 1) / kPage;               // <= 16
    SS_CHECK_OR(it.n_keys >= 0 && it.n_pages <= 32 && f_it.page0 >= 0 && f_it.page0 + it.n_pages <= P.total_node_pages &&
                    it.dec >= 0 && it.dec < P.caps.dec && it.g >= 0 && it.g < P.Hkv && f_it.q_src >= 0 &&
                    f_it.q_src < (P.q_src_offsets ? P.q_src_rows : P.total_q),
                &P.hdr->status, { it.valid = 0; return; });
    it.my_page = lane < it.n_pages ? P.node_pages[static_cast<int64_t>(f_it.page0) + lane] : 0;
    it.chunks = __ldcg(&P.dec_leaf_chunks[f_it.dec]);
    // B fragments of Q^T: thread (gid, tig) holds Q[row 8 nt + gid][dims 16 ks + 2 tig, + 1] and the same 8 dims on
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(P.q + (static_cast<int64_t>(f_it.q_src) * P.Hq + it.g * G) * kHeadDim);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int r = 8 * nt + gid;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        nq[nt][ks][0] = r < G ? __ldg(q0 + r * 64 + 8 * ks + tig) : 0u;
        nq[nt][ks][1] = r < G ? __ldg(q0 + r * 64 + 8 * ks + 4 + tig) : 0u;
      }
    }
  };

  Item cur, nxt;
  cur.valid = nxt.valid = 0;
  uint32_t n_issued = 0, n_cons = 0;
  int prod_pg = 0;                 // next page to request ...
  bool prod_in_next = false;       // ... of `nxt` (true) or of `cur`
  bool ok = true;

  // Requests one more page if the ring has room and an item with pages left is known (whole warp).
  auto issue_one = [&]() {
    if (n_issued - n_cons >= static_cast<uint32_t>(kStages)) return;
    if (!prod_in_next && prod_pg >= cur.n_pages) { prod_in_next = true; prod_pg = 0; }
    if (prod_in_next && (!nxt.valid || prod_pg >= nxt.n_pages)) return;
    int page = __shfl_sync(0xffffffffu, prod_in_next ? nxt.my_page : cur.my_page, prod_pg);
    SS_CHECK_OR(page >= 0 && page < P.num_pages, &P.hdr->status, page = 0);
    const int g = prod_in_next ? nxt.g : cur.g;
    const int stage = n_issued % kStages;
    if (lane == 0) {
      const int row = static_cast<int>((static_cast<int64_t>(page) * P.page_stride + static_cast<int64_t>(g) * P.head_stride) >> 7);
      uint64_t* bar = &full_bar[warp][stage];
      mbar_arrive_expect_tx(bar, kStageBytes);
      uint8_t* dst = ring_ptr + stage * kStageBytes;
      tma_load_4d(dst, &tmap_k, 0, 0, 0, row >> 3, bar);
      tma_load_4d(dst + kBlockBytes, &tmap_v, 0, 0, 0, row >> 3, bar);
    }
    ++n_issued;
    ++prod_pg;
  };

  // Per-lane address parts of the ldmatrix reads.  A landed block is [2 groups of 8 rows][2 halves of 64 dims][8 rows]
  // [128 B] with the 16-byte chunks of a row XOR-swizzled by the row.  K (not transposed): matrices (keys 0-7, c),
  // (keys 8-15, c), (keys 0-7, c+1), (keys 8-15, c+1) for the chunk pair of a 16-dim step; V (transposed): matrices
  // (keys 0-7, c), (keys 0-7, c+1), (keys 8-15, c), (keys 8-15, c+1) for the chunk pair of a 16-dim output tile.
  const int lm_i = lane >> 3, lm_r = lane & 7;
  const uint32_t k_lane = (lm_i & 1) * 2048 + lm_r * 128;
  const uint32_t v_lane = (lm_i >> 1) * 2048 + lm_r * 128;
  uint32_t k_ch[4], v_ch[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    k_ch[x] = static_cast<uint32_t>(((2 * x + (lm_i >> 1)) ^ lm_r) << 4);
    v_ch[x] = static_cast<uint32_t>(((2 * x + (lm_i & 1)) ^ lm_r) << 4);
  }

  if (n_items > 0) {
    fetch_claim();
    fetch_desc();
    fetch_finish(cur);
  }
  uint32_t qb[NT][8][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) { qb[nt][ks][0] = nq[nt][ks][0]; qb[nt][ks][1] = nq[nt][ks][1]; }
  int fetch_step = 3;              // 3: `nxt` is complete (or known to be absent)
  if (cur.valid) { fetch_claim(); fetch_step = 1; }

  while (cur.valid && ok) {
    for (int x = 0; x < kStages; ++x) issue_one();

    float o[8][NT][4];             // O^T: [16-dim tile][8-row group][dims gid, gid + 8 x columns 2 tig, 2 tig + 1]
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
    float m[NT][2], l[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { m[nt][0] = m[nt][1] = -INFINITY; l[nt][0] = l[nt][1] = 0.f; }

    for (int pg = 0; pg < cur.n_pages; ++pg) {
      const int stage = n_cons % kStages;
      if (!mbar_wait(&full_bar[warp][stage], (n_cons / kStages) & 1, abort_flag)) { ok = false; break; }
      const uint32_t kb = ring + stage * kStageBytes, vb = kb + kBlockBytes;
      const int valid = min(kPage, cur.n_keys - pg * kPage);       // keys of this page that exist
      if (valid < kPage) {
        // last page of the leaf: the rows past the length hold undefined data; clear them in V (their P is 0, but
        // 0 x NaN is NaN) - the scores of those keys are masked below
        for (int x = lane; x < (kPage - valid) * 16; x += 32) {
          const int r = valid + (x >> 4), ch = x & 15;
          *reinterpret_cast<uint4*>(ring_ptr + stage * kStageBytes + kBlockBytes + (r >> 3) * 2048 + (ch >> 3) * 1024 +
                                    (r & 7) * 128 + (ch & 7) * 16) = make_uint4(0, 0, 0, 0);
        }
        __syncwarp();
      }
      // ---- S^T = K Q^T ------------------------------------------------------------------------------------------------
      float s[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4(kb + (ks >> 2) * 1024 + k_lane + k_ch[ks & 3], a0, a1, a2, a3);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(s[nt], a0, a1, a2, a3, qb[nt][ks][0], qb[nt][ks][1]);
      }
      if (valid < kPage) {                                         // keys gid (s[.][0..1]) and gid + 8 (s[.][2..3])
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (gid >= valid) s[nt][0] = s[nt][1] = -INFINITY;
          if (gid + 8 >= valid) s[nt][2] = s[nt][3] = -INFINITY;
        }
      }
      // ---- online softmax per query column, over the 16 keys held by the 8 quad-groups --------------------------------
      uint32_t pb[NT][2];
      bool moved = false;
      float corr[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          float mx = fmaxf(s[nt][x], s[nt][2 + x]);
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          corr[nt][x] = 1.f;
          if (mx > m[nt][x] + lazy_raw) {                          // (also the first visible key: m = -inf)
            corr[nt][x] = ex2((m[nt][x] - mx) * c);                // ex2(-inf) = 0
            m[nt][x] = mx;
            moved = true;
          }
        }
        const float mc0 = m[nt][0] == -INFINITY ? 0.f : m[nt][0] * c, mc1 = m[nt][1] == -INFINITY ? 0.f : m[nt][1] * c;
        const float p00 = ex2(fmaf(s[nt][0], c, -mc0)), p01 = ex2(fmaf(s[nt][1], c, -mc1));   // key gid
        const float p10 = ex2(fmaf(s[nt][2], c, -mc0)), p11 = ex2(fmaf(s[nt][3], c, -mc1));   // key gid + 8
        l[nt][0] = l[nt][0] * corr[nt][0] + (p00 + p10);           // per-thread partial sums; reduced at the end
        l[nt][1] = l[nt][1] * corr[nt][1] + (p01 + p11);
        pb[nt][0] = movmatrix_trans(pack_bf16(p00, p01));          // -> P^T[keys 2 tig, 2 tig + 1][column gid]
        pb[nt][1] = movmatrix_trans(pack_bf16(p10, p11));          // -> the same for keys 8 ..
      }
      if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            o[mt][nt][0] *= corr[nt][0]; o[mt][nt][1] *= corr[nt][1];
            o[mt][nt][2] *= corr[nt][0]; o[mt][nt][3] *= corr[nt][1];
          }
      }
      // ---- O^T += V^T P^T -----------------------------------------------------------------------------------------------
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        uint32_t a0, a1, a2, a3;
        ldmatrix_x4_trans(vb + (mt >> 2) * 1024 + v_lane + v_ch[mt & 3], a0, a1, a2, a3);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16_16816(o[mt][nt], a0, a1, a2, a3, pb[nt][0], pb[nt][1]);
      }
      ++n_cons;
      // The stage is free: ldmatrix is warp-synchronous, so every lane's reads of it have been performed before the
      // copy that refills it is requested below.
      __syncwarp();
      if (fetch_step == 1) { fetch_desc(); fetch_step = 2; }
      else if (fetch_step == 2) { fetch_finish(nxt); fetch_step = 3; }
      issue_one();
    }
    if (!ok) break;
    ss::grid_dependency_wait();       // the tile kernel's partials are complete from here on (returns at once later)

    // ---- the item's normalised partial ---------------------------------------------------------------------------------
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        float v = l[nt][x];
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        l[nt][x] = v;
      }
    if (cur.chunks == 1) {
      // The leaf is this one item: nothing else will arrive for the (token, kv head), and the shared-node partials are
      // complete (the tile kernel ran before).  Fold them into the accumulator registers and write the final rows -
      // no partial of its own, no fence, no counter, no second pass over what was just written.
      int s0 = P.dec_slot_base[cur.dec], s1 = P.dec_slot_base[cur.dec + 1];
      const int64_t q_row = P.dec_tok[cur.dec];
      bool row_ok = true;
      SS_CHECK_OR(s0 >= 0 && s0 <= s1 && s1 <= P.caps.slots, &P.hdr->status, s1 = s0);
      SS_CHECK_OR(q_row >= 0 && q_row < P.total_q, &P.hdr->status, row_ok = false);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int q = 8 * nt + 2 * tig + x;
          const bool q_live = q < G;
          const int h = cur.g * G + (q_live ? q : 0);
          const float lq = l[nt][x];
          const float ms = m[nt][x] * P.scale;                     // (natural-log units; -inf if the leaf had no key)
          float big = lq > 0.f ? ms + __logf(lq) : -INFINITY;      // max of the log-sum-exps, own one first
          for (int s = s0; s < s1; ++s)
            if (s != cur.slot) big = fmaxf(big, __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h));
          const float a_own = lq > 0.f ? __expf(ms - big) : 0.f;   // weight of the unnormalised accumulator
          float den = a_own * lq;
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) { o[mt][nt][x] *= a_own; o[mt][nt][2 + x] *= a_own; }
          for (int s = s0; s < s1; ++s) {
            if (s == cur.slot) continue;
            const float ls = __ldcg(P.part_lse + static_cast<int64_t>(s) * P.Hq + h);
            const float w = ls == -INFINITY ? 0.f : __expf(ls - big);
            den += w;
            const float* src = P.part_o + (static_cast<int64_t>(s) * P.Hq + h) * kHeadDim + gid;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
              o[mt][nt][x] += w * __ldcg(src + 16 * mt);
              o[mt][nt][2 + x] += w * __ldcg(src + 16 * mt + 8);
            }
          }
          const float inv = den > 0.f ? 1.f / den : 0.f;
          // bf16 rows: lanes gid and gid ^ 1 hold neighbouring dims; the even one stores the pair of the lower 8 dims
          // of each 16-dim tile, the odd one the pair of the upper 8
          __nv_bfloat16* dst = P.out + (q_row * P.Hq + h) * kHeadDim + (gid & ~1) + ((gid & 1) ? 8 : 0);
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            const float lo = o[mt][nt][x] * inv, hi = o[mt][nt][2 + x] * inv;
            const float got = __shfl_xor_sync(0xffffffffu, (gid & 1) ? lo : hi, 4);
            const uint32_t pk = (gid & 1) ? pack_bf16(got, hi) : pack_bf16(lo, got);
            if (q_live && row_ok) *reinterpret_cast<uint32_t*>(dst + 16 * mt) = pk;
          }
          if (q_live && row_ok && gid == 0 && P.lse) P.lse[q_row * P.Hq + h] = den > 0.f ? big + __logf(den) : -INFINITY;
        }
    } else {
      bool slot_ok = true;
      SS_CHECK_OR(cur.slot >= 0 && cur.slot < P.caps.slots, &P.hdr->status, slot_ok = false);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int q = 8 * nt + 2 * tig + x;
          if (q >= G || !slot_ok) continue;
          const float lq = l[nt][x];
          const float inv = lq > 0.f ? 1.f / lq : 0.f;
          const int h = cur.g * G + q;
          float* dst = P.part_o + (static_cast<int64_t>(cur.slot) * P.Hq + h) * kHeadDim + gid;
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            dst[16 * mt] = o[mt][nt][x] * inv;
            dst[16 * mt + 8] = o[mt][nt][2 + x] * inv;
          }
          if (gid == 0) P.part_lse[static_cast<int64_t>(cur.slot) * P.Hq + h] = lq > 0.f ? m[nt][x] * P.scale + __logf(lq) : -INFINITY;
        }
      // ---- count the item; the last one of its (token, kv head) merges ---------------------------------------------------
      __syncwarp();
      int arrived = 0;
      if (lane == 0) {
        __threadfence();                                         // (cumulative: covers the stores of the other lanes)
        arrived = atomicAdd(&P.leaf_arrive[static_cast<int64_t>(cur.dec) * P.Hkv + cur.g], 1) + 1;
      }
      arrived = __shfl_sync(0xffffffffu, arrived, 0);
      if (arrived == cur.chunks) {
        __threadfence();
        for (int r0 = 0; r0 < G; r0 += 8) merge_rows8(P, cur.dec, cur.g * G + r0, min(8, G - r0), lane);
      }
    }

    // ---- next item --------------------------------------------------------------------------------------------------------
    if (fetch_step == 1) { fetch_desc(); fetch_step = 2; }
    if (fetch_step == 2) { fetch_finish(nxt); fetch_step = 3; }
    cur = nxt;
    nxt.valid = 0;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) { qb[nt][ks][0] = nq[nt][ks][0]; qb[nt][ks][1] = nq[nt][ks][1]; }
    if (prod_in_next) prod_in_next = false;                        // (the pages requested so far were the new item's)
    else prod_pg = 0;
    if (cur.valid) { fetch_claim(); fetch_step = 1; }
  }

  // ---- a wait ran out: let the copies in flight land before the shared memory is given back ----------------------------
  if (!ok) {
    while (n_cons < n_issued) {
      const int stage = n_cons % kStages;
      const long long t0 = clock64();
      while (!mbar_try_wait(&full_bar[warp][stage], (n_cons / kStages) & 1) && clock64() - t0 < 4000000LL) __nanosleep(200);
      ++n_cons;
    }
    if (lane == 0) set_status(&P.hdr->status, SS_ERR_TIMEOUT);
    ss::grid_dependency_wait();
    return;
  }
  ss::grid_dependency_wait();         // (every thread, before the sweeps below and before the kernel ends)
  if (!plan_ok) return;

  // ---- decode tokens without a private leaf (empty or shared): their partials all come from the tile kernel -------------
  const int64_t warps = static_cast<int64_t>(gridDim.x) * WARPS;
  const int64_t w0 = static_cast<int64_t>(blockIdx.x) * WARPS + warp;
  const int64_t n_tok_heads = static_cast<int64_t>(P.hdr->n_dec) * P.Hkv;
  for (int64_t w = w0; w < n_tok_heads; w += warps) {
    const int d = static_cast<int>(w / P.Hkv), g = static_cast<int>(w % P.Hkv);
    if (P.dec_leaf_chunks[d] != 0) continue;
    for (int r0 = 0; r0 < G; r0 += 8) merge_rows8(P, d, g * G + r0, min(8, G - r0), lane);
  }
  // ---- rows of GENERIC paths -------------------------------------------------------------------------------------------
  if (P.hdr->n_generic_rows > 0) generic_rows(P, w0, warps, lane);
  SS_STAMP_END(P.hdr, 5);
}

}  // namespace leafs

// False if the pool layout rules the streaming kernel out (the caller then takes the register-staged kernel and the
// separate merge launch).
bool leaf_stream_supported(const Params& P) {
  return P.page_stride % 1024 == 0 && P.head_stride % 1024 == 0 && P.G <= 16;
}

template <int NT, int WARPS, int STAGES>
static int32_t launch_variant(const Params& P, cudaStream_t st, int sm_count, const CUtensorMap& tk, const CUtensorMap& tv) {
  using namespace leafs;
  using C = Cfg<NT, WARPS, STAGES>;
  static bool configured[kDeviceSlots] = {false};
  const int dev_slot = current_device_slot();
  if (dev_slot < 0 || !configured[dev_slot]) {
    if (cudaFuncSetAttribute(leaf_stream_kernel<NT, WARPS, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmem) != cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    if (dev_slot >= 0) configured[dev_slot] = true;
  }
  SS_LAUNCH((leaf_stream_kernel<NT, WARPS, STAGES>), sm_count, WARPS * 32, C::kSmem, st, tk, tv, P);
  return SS_OK;
}

int32_t launch_leaf_stream(const Params& P, cudaStream_t st, int sm_count) {
  const int64_t rows = ((P.num_pages > 0 ? P.num_pages - 1 : 0) * P.page_stride + (P.Hkv - 1) * P.head_stride) / 128 + kPage;
  if (rows >= 0x7fffffffLL) return SS_ERR_UNSUPPORTED;
  CUtensorMap tk, tv;
  if (!tmap::encode_kv_block_bf16(&tk, P.k_pool, static_cast<uint64_t>(rows)) ||
      !tmap::encode_kv_block_bf16(&tv, P.v_pool, static_cast<uint64_t>(rows)))
    return SS_ERR_CUDA;
  if (P.G > 8) return launch_variant<2, 8, 3>(P, st, sm_count, tk, tv);
  return launch_variant<1, 12, 2>(P, st, sm_count, tk, tv);
}

}  // namespace attn
}  // namespace ss
