// Tensor-core tile kernel of ss_tree_attention (tcgen05 + TMEM + TMA), for the planner's tile items:
//   * stacked items: up to 128 stacked rows (decode tokens below a shared node x GQA group) against that node's
//     keys - the shared prefix / branch KV tile is staged in shared memory once for all paths below the node;
//   * chain items: up to 128 rows (tokens of one verification step x GQA group) against the path's whole key chain
//     root -> leaf, causal inside the step.
//
// One CTA works on one item at a time (items are fetched from a global counter) and two CTAs share an SM, so one
// CTA's softmax overlaps the other's MMAs.  Warp roles:
//   warps 0-3  softmax + epilogue, one query row per thread = one TMEM lane
//   warp 4     TMA producer: paged K / V boxes (one 16-token page x 64 dims each, 128-byte swizzle) into a
//              2-stage ring, separate full/empty barriers for K and V
//   warp 5     lane 0 issues the MMAs: S[b] = Q K^T (M128 N64 K16 x 8), O += P[b] V (M128 N128 K16 x 4, P in TMEM,
//              V MN-major);
//              the warp also owns the TMEM allocation (256 columns: two S buffers + O)
// Per 64-key tile:  QK^T of tile j+1 is issued before PV of tile j, so the tensor pipe works on the next scores
// while the softmax warps turn S[j] into P[j].  P (bf16) is written back into the TMEM columns of its own S buffer
// and is the A operand of the PV product straight from TMEM, so it never touches shared memory.  The exponentials
// use a lazily updated reference maximum, so the O accumulator in TMEM is rescaled only when a row maximum jumps
// by more than 2^8.  Softmax runs in the exp2 domain with the scale folded in.
// Every mbarrier wait is bounded; on expiry the CTA raises its abort flag, all roles fall through to the item-end
// barrier, the CTA frees its TMEM and the kernel records SS_ERR_TIMEOUT.
#include "attn_plan.cuh"
#include "umma.cuh"

namespace ss {
namespace attn {

using namespace umma;

constexpr int kUmmaThreads = 192;
constexpr int kStages = 2;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColO = 128;
constexpr float kLazyLog2 = 8.0f;              // the reference maximum moves only when exceeded by 2^8
constexpr int kOffQ = 0;                       // [2 halves][128 rows][128 B]
constexpr int kOffK = 32768;                   // kStages x [2 halves][64 rows][128 B]
constexpr int kOffV = kOffK + kStages * 16384;
constexpr int kOffCtrl = kOffV + kStages * 16384;
constexpr int kUmmaSmem = kOffCtrl + 1024;

struct Ctrl {
  // Parity waits are only safe when the waiter is never two completions away from the barrier's phase, hence:
  // p_full is per S/P buffer (the softmax warps may run one tile ahead of the MMA thread), pv_done is waited only
  // for the previous tile (it cannot lag further once S of the current tile exists), o_final fires once per item.
  uint64_t q_full, k_full[kStages], v_full[kStages], k_empty[kStages], v_empty[kStages], s_full[2], p_full[2], pv_done,
      o_final;
  uint32_t tmem_slot;
  int abort_flag;
  int item_idx;
  int n_seg;
  int seg_first_page[SS_MAX_DEPTH + 1];
  long long seg_page_off[SS_MAX_DEPTH];
};
static_assert(sizeof(Ctrl) <= 1024, "control block must fit its kilobyte");

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct ItemView {
  int node, tok0, n_tok, kind, g, kv_begin, kv_end, limit0, slot_off, src0, n_tiles;
};

__device__ __forceinline__ ItemView view(const TileItem& it) {
  ItemView v;
  v.node = it.node; v.tok0 = it.tok0; v.n_tok = it.n_tok;
  v.kind = it.kind_g >> 16; v.g = it.kind_g & 0xffff;
  v.kv_begin = it.kv_begin; v.kv_end = it.kv_end; v.limit0 = it.limit0; v.slot_off = it.slot_off;
  v.src0 = it.src0;
  v.n_tiles = v.kv_end > v.kv_begin ? (v.kv_end - v.kv_begin + kKvTile - 1) / kKvTile : 0;
  return v;
}

__global__ void __launch_bounds__(kUmmaThreads, 2)
tile_items_umma_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                       const Params P) {
  ss::grid_dependency_enter_then_release();   // (the leaf kernel behind this one starts without waiting for it)
  extern __shared__ __align__(1024) uint8_t smem[];
  Ctrl& C = *reinterpret_cast<Ctrl*>(smem + kOffCtrl);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &C.abort_flag;

  if (tid == 0) {
    C.abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
    mbar_init(&C.q_full, 128);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&C.k_full[s], 1); mbar_init(&C.v_full[s], 1);
      mbar_init(&C.k_empty[s], 1); mbar_init(&C.v_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(&C.s_full[b], 1); mbar_init(&C.p_full[b], 128); }
    mbar_init(&C.pv_done, 1);
    mbar_init(&C.o_final, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmap_k);
    prefetch_tensormap(&tmap_v);
  }
  if (warp == 5) tmem_alloc(&C.tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = C.tmem_slot;
  const int n_items = P.hdr->n_tile_items;
  const int G = P.G;
  const float cl2 = P.scale_log2;
  const float lazy_raw = kLazyLog2 / cl2;   // the lazy-rescale threshold in raw score units

  uint32_t g_tile = 0;      // tiles this CTA has processed (identical in every role)
  uint32_t q_uses = 0;      // items with at least one tile

  for (;;) {
    if (tid == 0) {
      int e = -1;
      if (P.hdr->status == SS_OK && !C.abort_flag) e = atomicAdd(&P.hdr->tile_counter, 1);
      C.item_idx = e;
    }
    __syncthreads();
    const int e = C.item_idx;
    if (e < 0 || e >= n_items) break;
    const ItemView it = view(P.tile_items[e]);
    const int n_tiles = it.n_tiles;

    if (warp < 4) {
      // =================================================== softmax + epilogue ==================================
      const int row = tid;
      const int i = row / G, hl = row - i * G;
      const bool row_valid = i < it.n_tok;
      const int h = it.g * G + hl;
      int64_t q_row = 0, q_src = 0;                               // output row / row of q holding the query
      int dec = 0;
      if (row_valid) {
        if (it.kind == kItemChain) { q_row = it.tok0 + i; q_src = it.src0 + i; }
        else { dec = it.tok0 + i; q_row = P.dec_tok[dec]; q_src = P.dec_src[dec]; }
      }
      const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
      float m = -INFINITY, l = 0.f;
      bool ok = true;
      if (n_tiles > 0) {
        // ---- Q rows into the UMMA operand layout ---------------------------------------------------------------
        {
          const uint4* src = reinterpret_cast<const uint4*>(P.q + (q_src * P.Hq + h) * kHeadDim);
#pragma unroll
          for (int ch = 0; ch < 16; ++ch) {
            const uint4 v = row_valid ? __ldg(src + ch) : make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(smem + kOffQ + (ch >> 3) * 16384 + sw128_offset(row, ch & 7)) = v;
          }
          fence_proxy_async_smem();
          mbar_arrive(&C.q_full);
        }
        int limit_row = (it.kind == kItemChain) ? it.limit0 + i : it.limit0;
        if (limit_row > it.kv_end) limit_row = it.kv_end;
        for (int j = 0; j < n_tiles; ++j) {
          const uint32_t gj = g_tile + j;
          const int b = gj & 1;
          ok = mbar_wait(&C.s_full[b], (gj >> 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          uint32_t sr[64];
          tmem_ld32(tmem + lane_base + b * 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
          tmem_ld32(tmem + lane_base + b * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
          tmem_wait_ld();

          const int pos0 = it.kv_begin + j * kKvTile;
          const int nvis = limit_row - pos0;                      // visible columns of this tile for this row
          if (!__all_sync(0xffffffffu, nvis >= kKvTile)) {        // causal tail or end of the source: mask
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (c >= nvis) sr[c] = 0xff800000u;                 // -inf
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 64; c += 4) {
#pragma unroll
            for (int x = 0; x < 4; ++x) mx4[x] = fmaxf(mx4[x], __uint_as_float(sr[c + x]));
          }
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          // Lazy reference maximum: exponentials are taken relative to m (not the running maximum); m only moves
          // when the tile's maximum exceeds it by more than 2^kLazyLog2, so P stays <= 2^kLazyLog2 and the O
          // accumulator in TMEM rarely needs rescaling.  out = O / l and lse = m*scale + ln l hold for any m.
          const bool move = mx > m + lazy_raw;                    // also true for the first visible key (m = -inf)
          float alpha = 1.f;
          if (move) {
            alpha = ex2((m - mx) * cl2);                          // 0 when the row had no visible key so far
            m = mx;
            l *= alpha;
          }
          const float mc = m == -INFINITY ? 0.f : m * cl2;
          float sum4[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t pr[32];
#pragma unroll
          for (int c = 0; c < 64; c += 2) {
            const float p0 = ex2(__uint_as_float(sr[c]) * cl2 - mc);
            const float p1 = ex2(__uint_as_float(sr[c + 1]) * cl2 - mc);
            sum4[(c >> 1) & 3] += p0 + p1;
            __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            pr[c >> 1] = *reinterpret_cast<uint32_t*>(&pk);
          }
          l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);

          if (__any_sync(0xffffffffu, move && j > 0)) {           // rescale O (warp-collective TMEM access)
            ok = mbar_wait(&C.pv_done, (gj - 1) & 1, abort_flag); // PV of the previous tile must have landed in O
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < kHeadDim; c0 += 64) {
              uint32_t o0[32], o1[32];
              tmem_ld32(tmem + lane_base + kColO + c0, o0);
              tmem_ld32(tmem + lane_base + kColO + c0 + 32, o1);
              tmem_wait_ld();
#pragma unroll
              for (int x = 0; x < 32; ++x) {
                o0[x] = __float_as_uint(__uint_as_float(o0[x]) * alpha);
                o1[x] = __float_as_uint(__uint_as_float(o1[x]) * alpha);
              }
              tmem_st32(tmem + lane_base + kColO + c0, o0);
              tmem_st32(tmem + lane_base + kColO + c0 + 32, o1);
            }
            tmem_wait_st();
          }
          // ---- last tile of a source that ends inside a page / inside the tile: zero the V rows past the end ---
          const int n_keys = min(kKvTile, it.kv_end - pos0);
          if (n_keys < kKvTile) {
            const int s = gj % kStages;
            ok = mbar_wait(&C.v_full[s], (gj / kStages) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            uint8_t* vs = smem + kOffV + s * 16384;
            const int n_chunks = (kKvTile - n_keys) * 16;         // 16-byte chunks to clear (both halves)
            for (int x = tid; x < n_chunks; x += 128) {
              const int r = n_keys + (x >> 4), cc = x & 15;
              *reinterpret_cast<uint4*>(vs + (cc >> 3) * 8192 + r * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          // ---- P (bf16 pairs) over the first 32 columns of its own S buffer: the A operand of PV, read from TMEM ------
          tmem_st32(tmem + lane_base + b * 64, pr);
          tmem_wait_st();
          if (n_keys < kKvTile) fence_proxy_async_smem();         // the V rows cleared above
          tc_fence_before();
          mbar_arrive(&C.p_full[b]);
        }
        if (ok) {
          ok = mbar_wait(&C.o_final, q_uses & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          tc_fence_after();
        }
      }
      // ---- epilogue --------------------------------------------------------------------------------------------------
      if (ok) {
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const float lse = l > 0.f ? m * P.scale + __logf(l) : -INFINITY;
        const bool final_out = it.slot_off < 0;
        const int64_t slot = final_out ? 0 : static_cast<int64_t>(row_valid ? P.dec_slot_base[dec] : 0) + it.slot_off;
        bool store_ok = true;
        SS_CHECK_OR(!row_valid || (final_out ? (q_row >= 0 && q_row < P.total_q) : (slot >= 0 && slot < P.caps.slots)),
                    &P.hdr->status, store_ok = false);
#pragma unroll
        for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
          uint32_t orow[32];
          __syncwarp();                                         // the TMEM load below is warp-collective
          if (n_tiles > 0) {
            tmem_ld32(tmem + lane_base + kColO + c0, orow);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int x = 0; x < 32; ++x) orow[x] = 0u;
          }
          if (!row_valid || !store_ok) continue;
          if (final_out) {
            uint4* dst = reinterpret_cast<uint4*>(P.out + (q_row * P.Hq + h) * kHeadDim + c0);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              uint32_t w[4];
#pragma unroll
              for (int y = 0; y < 4; ++y) {
                __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(orow[8 * x + 2 * y]) * inv,
                                                          __uint_as_float(orow[8 * x + 2 * y + 1]) * inv);
                w[y] = *reinterpret_cast<uint32_t*>(&pk);
              }
              dst[x] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          } else {
            float4* dst = reinterpret_cast<float4*>(P.part_o + (slot * P.Hq + h) * kHeadDim + c0);
#pragma unroll
            for (int x = 0; x < 8; ++x)
              dst[x] = make_float4(__uint_as_float(orow[4 * x]) * inv, __uint_as_float(orow[4 * x + 1]) * inv,
                                   __uint_as_float(orow[4 * x + 2]) * inv, __uint_as_float(orow[4 * x + 3]) * inv);
          }
        }
        if (row_valid && store_ok) {
          if (final_out) { if (P.lse) P.lse[q_row * P.Hq + h] = lse; }
          else P.part_lse[slot * P.Hq + h] = lse;
        }
      }
    } else if (warp == 4) {
      // =================================================== TMA producer ========================================
      if (n_tiles > 0) {
        if (lane == 0) {
          int n_seg = 0;
          if (it.kind == kItemChain) {
            int chain[SS_MAX_DEPTH];
            int d = 0;
            for (int a = it.node; a >= 0 && d < SS_MAX_DEPTH; a = P.node_parent[a]) chain[d++] = a;
            int first = 0;
            for (int c = d - 1; c >= 0; --c) {
              const int n = chain[c];
              const int np = (P.node_kv_len[n] + kPage - 1) / kPage;
              if (np == 0) continue;
              C.seg_first_page[n_seg] = first;
              C.seg_page_off[n_seg] = P.node_page_offsets[n];
              first += np;
              ++n_seg;
            }
            C.seg_first_page[n_seg] = first;
          } else {
            C.seg_first_page[0] = 0;
            C.seg_page_off[0] = P.node_page_offsets[it.node];
            C.seg_first_page[1] = 0x7fffffff;
            n_seg = 1;
          }
          C.n_seg = n_seg;
        }
        __syncwarp();
        const int n_seg = C.n_seg;
        bool ok = true;
        // page of tile j handled by this lane -> row coordinate of its (page, kv head) block in the pool
        auto page_coord = [&](int j) -> int {
          const int pos0 = it.kv_begin + j * kKvTile;
          const int n_pages = (min(kKvTile, it.kv_end - pos0) + kPage - 1) / kPage;
          if (j >= n_tiles || lane >= n_pages) return 0;
          const int vp = pos0 / kPage + lane;
          int d = 0;
          while (d + 1 < n_seg && vp >= C.seg_first_page[d + 1]) ++d;
          int64_t phys = P.node_pages[C.seg_page_off[d] + (vp - C.seg_first_page[d])];
          SS_CHECK_OR(phys >= 0 && phys < P.num_pages, &P.hdr->status, phys = 0);
          return static_cast<int>((phys * P.page_stride + static_cast<int64_t>(it.g) * P.head_stride) >> 7);
        };
        int next_coord = page_coord(0);
        for (int j = 0; j < n_tiles && ok; ++j) {
          const uint32_t gj = g_tile + j;
          const int s = gj % kStages;
          const uint32_t u = gj / kStages;
          const int pos0 = it.kv_begin + j * kKvTile;
          const int n_keys = min(kKvTile, it.kv_end - pos0);
          const int n_pages = (n_keys + kPage - 1) / kPage;
          const int coord_y = next_coord;
          next_coord = page_coord(j + 1);                         // in flight while this tile's slots are awaited
          // K
          if (u > 0) ok = mbar_wait(&C.k_empty[s], (u - 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) mbar_arrive_expect_tx(&C.k_full[s], static_cast<uint32_t>(n_pages) * 4096u);
          __syncwarp();
          if (lane < n_pages) {
            uint8_t* dst = smem + kOffK + s * 16384 + lane * 2048;
            tma_load_2d(dst, &tmap_k, 0, coord_y, &C.k_full[s]);
            tma_load_2d(dst + 8192, &tmap_k, 64, coord_y, &C.k_full[s]);
          }
          // V
          if (u > 0) ok = mbar_wait(&C.v_empty[s], (u - 1) & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          if (lane == 0) mbar_arrive_expect_tx(&C.v_full[s], static_cast<uint32_t>(n_pages) * 4096u);
          __syncwarp();
          if (lane < n_pages) {
            uint8_t* dst = smem + kOffV + s * 16384 + lane * 2048;
            tma_load_2d(dst, &tmap_v, 0, coord_y, &C.v_full[s]);
            tma_load_2d(dst + 8192, &tmap_v, 64, coord_y, &C.v_full[s]);
          }
        }
      }
    } else if (lane == 0 && n_tiles > 0) {
      // =================================================== MMA issuer ==========================================
      constexpr uint32_t idesc_qk = instr_desc_bf16(128, kKvTile, false);
      constexpr uint32_t idesc_pv = instr_desc_bf16(128, kHeadDim, true);
      // descriptors of the operand tiles at stage 0 / K-step 0; every MMA below derives its own with one add
      const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + kOffQ), 0, 1024);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + kOffK), 0, 1024);
      const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + kOffV), 8192, 1024);
      bool ok = mbar_wait(&C.q_full, q_uses & 1, abort_flag);
      auto issue_qk = [&](int j) -> bool {
        const uint32_t gj = g_tile + j;
        const int s = gj % kStages, b = gj & 1;
        // S[b] / P[b] of tile gj-2 is free: PV(gj-2) was issued earlier by this thread and MMAs execute in order
        if (!mbar_wait(&C.k_full[s], (gj / kStages) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint64_t k_desc = smem_desc_advance(k_desc0, static_cast<uint32_t>(s) * 16384u);
        const uint32_t d_tmem = tmem + b * 64;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t ad = smem_desc_advance(q_desc0, (kk >> 2) * 16384 + (kk & 3) * 32);
          const uint64_t bd = smem_desc_advance(k_desc, (kk >> 2) * 8192 + (kk & 3) * 32);
          mma_bf16_ss(d_tmem, ad, bd, idesc_qk, kk > 0 ? 1u : 0u);
        }
        mma_commit(&C.k_empty[s]);
        mma_commit(&C.s_full[b]);
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int j = 0; j < n_tiles && ok; ++j) {
        if (j + 1 < n_tiles) ok = issue_qk(j + 1);
        if (!ok) break;
        const uint32_t gj = g_tile + j;
        const int s = gj % kStages, b = gj & 1;
        ok = mbar_wait(&C.v_full[s], (gj / kStages) & 1, abort_flag) &&
             mbar_wait(&C.p_full[b], (gj >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t v_desc = smem_desc_advance(v_desc0, static_cast<uint32_t>(s) * 16384u);
        const uint32_t o_tmem = tmem + kColO, p_tmem = tmem + b * 64;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          mma_bf16_ts(o_tmem, p_tmem + kk * 8, smem_desc_advance(v_desc, kk * 2048), idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
        mma_commit(&C.v_empty[s]);
        mma_commit(&C.pv_done);
        if (j + 1 == n_tiles) mma_commit(&C.o_final);
      }
    }
    // ---- item end: every role meets here, so the next item starts from a drained pipeline --------------------
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    g_tile += n_tiles;
    if (n_tiles > 0) ++q_uses;
  }

  // ---- teardown --------------------------------------------------------------------------------------------------
  __syncthreads();
  if (C.abort_flag) {
    if (tid == 0) set_status(&P.hdr->status, SS_ERR_TIMEOUT);
    const long long t0 = clock64();                 // let copies / MMAs that are still in flight land
    while (clock64() - t0 < 4000000LL) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) tmem_dealloc(tmem, kTmemCols);
}

int g_tile_kernel_occupancy = 0;   // CTAs per SM reported by the occupancy query (diagnostics)

int32_t launch_tile_items_umma(const Params& P, cudaStream_t st, int sm_count) {
  static bool configured[kDeviceSlots] = {false};     // the attributes belong to the (function, device) pair
  constexpr int ctas_per_sm = 2;                      // TMEM: 2 x 256 columns per SM; extra CTAs simply queue
  const int dev_slot = current_device_slot();
  if (dev_slot < 0 || !configured[dev_slot]) {
    if (cudaFuncSetAttribute(tile_items_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    // two CTAs per SM need the largest shared-memory carve-out (2 x 113 KB + 2 KB reserved = 228 KB)
    if (cudaFuncSetAttribute(tile_items_umma_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared) != cudaSuccess)
      (void)cudaGetLastError();
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, tile_items_umma_kernel, kUmmaThreads, kUmmaSmem) !=
            cudaSuccess || occ < 1) {
      (void)cudaGetLastError();
      occ = 1;
    }
    g_tile_kernel_occupancy = occ;
    if (dev_slot >= 0) configured[dev_slot] = true;
  }
  const int64_t rows = ((P.num_pages > 0 ? P.num_pages - 1 : 0) * P.page_stride + (P.Hkv - 1) * P.head_stride) / 128 + kPage;
  if (rows >= 0x7fffffffLL) return SS_ERR_UNSUPPORTED;
  CUtensorMap tk, tv;
  if (!tmap::encode_2d_bf16(&tk, P.k_pool, kHeadDim, static_cast<uint64_t>(rows), kHeadDim * 2, kPage) ||
      !tmap::encode_2d_bf16(&tv, P.v_pool, kHeadDim, static_cast<uint64_t>(rows), kHeadDim * 2, kPage))
    return SS_ERR_CUDA;
  SS_LAUNCH(tile_items_umma_kernel, sm_count * ctas_per_sm, kUmmaThreads, kUmmaSmem, st, tk, tv, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss

extern "C" int32_t ss_debug_tile_kernel_occupancy(void) { return ss::attn::g_tile_kernel_occupancy; }
