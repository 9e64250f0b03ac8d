// Tensor-core tile kernel of ss_tree_attention, deep-pipeline version (tcgen05 + TMEM + TMA): one CTA per SM that owns
// all 512 TMEM columns and works on 128-key tiles.  Same items and the same arithmetic as the two-CTAs-per-SM kernel in
// attn_umma.cu (a 64-key tile there); what differs follows from three measurements on this part:
//   * an SM retires one tcgen05 instruction (MMA or commit) per ~50 clocks whatever its shape, and a 64-key tile costs
//     17 of them: with 128-key tiles every MMA is M128 x N128 x K16 (64 clocks of math) and the count per key halves;
//   * an ex2 holds an SM sub-partition for 8 clocks and every other instruction of the softmax loop ADDS to that (the
//     pipes do not overlap in issue), so the loop works on packed fp32 pairs, takes the row maximum from a sample of
//     the columns inside the exponential loop, and uses a reference maximum that lags one tile behind;
//   * a score buffer is recycled only when the P V product that read it has completed, so with two buffers the chain
//     Q K^T -> softmax -> P V of one tile bounds the next but one: three S/P buffers (128 columns each) + O (128
//     columns) fill the TMEM exactly, Q stays in shared memory.
// Roles: warps 0-3 softmax + epilogue (one query row per thread = one TMEM lane); warp 4 streams K tiles and warp 5
// V tiles through TMA (3 and 2 stages of 32 KB); warp 6 lane 0 issues S[b] = Q K^T (8 MMAs per tile), warp 7 lane 0
// issues O += P[b] V (8 MMAs, P read from TMEM where it overwrote the first 64 columns of S[b], V MN-major), lane 1
// of warp 7 fetches the NEXT item while this one runs: the producers then load its first K / V tiles and its Q rows
// (a 3-D TMA box for a chain item, issued by the K producer; cp.async of the gathered rows of a stacked item by the
// V producer warp) into the second Q buffer before the current item has drained.  The softmax warps do nothing but
// the softmax and the epilogue: every other duty that sat in their loop cost more than it looked.
// Every wait is bounded; on expiry the CTA raises its abort flag, all roles fall through to the item-end barrier,
// the CTA frees its TMEM and the kernel records SS_ERR_TIMEOUT.
#include "attn_plan.cuh"
#include "umma.cuh"

namespace ss {
namespace attn {

using namespace umma;

namespace deep {

constexpr int kSoftmaxWarps = 4;
constexpr int kUmmaThreads = (kSoftmaxWarps + 4) * 32;
constexpr int kTile = 128;                     // keys per tile (two of the planner's 64-key tiles)
constexpr int kStageBytes = kTile * 256;       // one K or V tile: [2 halves of 64 dims][kTile rows][128 B]
constexpr int kStagesK = 3;
constexpr int kStagesV = 2;                    // V is consumed a softmax later than K: two stages are enough
constexpr int kRing = 3;                       // S/P buffers
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                  // kRing x kTile columns
constexpr uint32_t kColO = kRing * kTile;      // 128 columns
constexpr float kLazyLog2 = 8.0f;              // the reference maximum moves only when exceeded by 2^8
constexpr float kJumpLog2 = 40.0f;             // exponentials may exceed the reference by at most 2^40 (+2^8 lag)
constexpr int kOffQ = 0;                       // 2 buffers (this item / next item) x [2 halves of 64 dims][128 rows][128 B]
constexpr int kOffK = 65536;
constexpr int kOffV = kOffK + kStagesK * kStageBytes;
constexpr int kUmmaSmem = kOffV + kStagesV * kStageBytes;   // + the control block in static shared memory

struct Ctrl {
  // All per-buffer barriers are indexed by tile number modulo the ring / stage count and waited with the parity of
  // (tile number / count); a waiter is never two completions away from its barrier (see the role loops).
  uint64_t q_full, q_full_tma, k_full[kStagesK], v_full[kStagesV], k_empty[kStagesK], v_empty[kStagesV], s_full[kRing],
      p_full[kRing], pv_done[kRing], o_final, item_ready[2];
  uint32_t tmem_slot;
  int abort_flag;
  // Items are fetched one ahead: while item k (slot k & 1) is processed, a spare lane takes item k+1 from the global
  // counter and copies its descriptor into the other slot, so that the producers can start its K / V tiles and the
  // softmax warps its Q rows before item k has drained.
  int item_e[2];
  TileItem item[2];
  alignas(16) int page_coord[2][32];             // row coordinates of the pages of four tiles, one block per producer warp
  int n_seg[2];                                  // page-segment tables of the chain, one copy per producer warp
  int seg_first_page[2][SS_MAX_DEPTH + 1];
  long long seg_page_off[2][SS_MAX_DEPTH];
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- packed fp32 pairs (one issue slot for two values) and the three-input maximum ---------------------------------
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float a, float b) { f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ float max3(float a, float b, float c) { float r; asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c)); return r; }
__device__ __forceinline__ uint32_t pack_bf16_rn(float a, float b) {
  __nv_bfloat162 pk = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&pk);
}

// 32-byte store (a whole sector per lane: the epilogue writes one row per thread, so a 16-byte store leaves half of
// every sector for a second transaction).  `p` must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e, uint32_t f,
                                              uint32_t g, uint32_t h) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e),
               "r"(f), "r"(g), "r"(h) : "memory");
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
  v.n_tiles = v.kv_end > v.kv_begin ? (v.kv_end - v.kv_begin + kTile - 1) / kTile : 0;
  return v;
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
tile_items_umma_deep_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                            const __grid_constant__ CUtensorMap tmap_q, const Params P) {
  ss::grid_dependency_enter();
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctrl C;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &C.abort_flag;

  if (tid == 0) {
    C.abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
    mbar_init(&C.q_full, 1);                        // stacked items: the V producer warp copies the (gathered) rows
    mbar_init(&C.q_full_tma, 1);                    // chain items: one TMA box pair
    for (int s = 0; s < kStagesK; ++s) { mbar_init(&C.k_full[s], 1); mbar_init(&C.k_empty[s], 1); }
    for (int s = 0; s < kStagesV; ++s) { mbar_init(&C.v_full[s], 1); mbar_init(&C.v_empty[s], 1); }
    mbar_init(&C.item_ready[0], 1);
    mbar_init(&C.item_ready[1], 1);
    for (int b = 0; b < kRing; ++b) {
      mbar_init(&C.s_full[b], 1); mbar_init(&C.p_full[b], kSoftmaxWarps * 32); mbar_init(&C.pv_done[b], 1);
    }
    mbar_init(&C.o_final, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmap_k);
    prefetch_tensormap(&tmap_v);
    prefetch_tensormap(&tmap_q);
  }
  for (int x = tid; x < 65536 / 16; x += kUmmaThreads) reinterpret_cast<uint4*>(smem + kOffQ)[x] = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  if (warp == kSoftmaxWarps) tmem_alloc(&C.tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = C.tmem_slot;
  const int n_items = P.hdr->n_tile_items;
  const int G = P.G;
  const float cl2 = P.scale_log2;
  const float lazy_raw = kLazyLog2 / cl2;   // the lazy-rescale threshold in raw score units
  const float jump_sum = exp2f(kJumpLog2);  // a tile whose exponentials sum to more than this takes the exact path

  uint32_t g_tile = 0;      // tiles this CTA has processed (identical in every role)
  uint32_t q_uses = 0;      // items with at least one tile
  uint32_t q_uses_tma = 0;  // ... of them chain items (their Q arrives through TMA and q_full_tma)
  uint32_t item_seq = 0;    // items this CTA has started
  int n_prefetched = 0;     // producer warps: tiles of the current item that were issued during the previous one
  int prod_stage = 0;       // producer warps: ring stage of the next tile to issue, and how often the ring has wrapped
  uint32_t prod_wraps = 0;  //   (kept as counters: a modulo by a stage count that differs per warp is a division per tile)

  // Takes the next item from the global counter into slot `dst` (one thread).
  auto fetch_item = [&](int dst) {
    int e = -1;
    if (P.hdr->status == SS_OK && !C.abort_flag) e = atomicAdd(&P.hdr->tile_counter, 1);
    if (e >= 0 && e < n_items) C.item[dst] = P.tile_items[e];
    C.item_e[dst] = e;
    __threadfence_block();
    mbar_arrive(&C.item_ready[dst]);
  };
  // Stacked items: one producer warp starts the asynchronous copy of item `v`'s (gathered) Q rows into Q buffer `buf`
  // (UMMA K-major layout with the 128-byte swizzle; rows past the item's last one are zero-filled).  The softmax
  // warps used to do this inside their tile loop, where the dependent load of the row index and the hundred
  // instructions of the copy cost each of them about 1400 clocks per item.
  auto q_gather_start = [&](const ItemView& v, int buf) {
    const uint32_t dst0 = smem_u32(smem + kOffQ + buf * 32768);
#pragma unroll 1
    for (int row = lane; row < 128; row += 32) {
      const int i = row / G, hl = row - i * G;
      const bool row_valid = i < v.n_tok;
      int64_t q_src = 0;
      if (row_valid) q_src = P.dec_src[v.tok0 + i];
      const char* src = reinterpret_cast<const char*>(P.q + (q_src * P.Hq + (v.g * G + hl)) * kHeadDim);
      const uint32_t n_src = row_valid ? 16u : 0u;               // 0 source bytes: the 16 destination bytes are zeroed
#pragma unroll
      for (int ch = 0; ch < 16; ++ch)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst0 + (ch >> 3) * 16384 + sw128_offset(row, ch & 7)),
                     "l"(src + ch * 16), "r"(n_src) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  // Chain items: the Q rows are tokens [src0, src0 + tokens per tile) x the G heads of the group x 128 dims, a box of
  // the query tensor (one thread; rows of the box past the item's tokens belong to other paths or are zero-filled:
  // finite either way, and never written out).
  auto q_tma_start = [&](const ItemView& v, int buf) {
    uint8_t* dst = smem + kOffQ + buf * 32768;
    mbar_arrive_expect_tx(&C.q_full_tma, static_cast<uint32_t>(2 * 128 * G * P.tok_per_tile));
    tma_load_3d(dst, &tmap_q, 0, v.g * G, v.src0, &C.q_full_tma);
    tma_load_3d(dst + 16384, &tmap_q, 64, v.g * G, v.src0, &C.q_full_tma);
  };

  if (tid == 0) fetch_item(0);
  __syncthreads();
  bool q_pending = false;   // V producer warp: a gather of the coming item's Q rows is under way
  if (warp == kSoftmaxWarps + 1) {                               // Q of a first stacked item
    if (__all_sync(0xffffffffu, mbar_wait(&C.item_ready[0], 0, abort_flag))) {
      const int e0 = C.item_e[0];
      if (e0 >= 0 && e0 < n_items) {
        const ItemView v0 = view(C.item[0]);
        if (v0.n_tiles > 0 && v0.kind != kItemChain) { q_gather_start(v0, 0); q_pending = true; }
      }
    }
  }

  if (tid == kSoftmaxWarps * 32 && mbar_wait(&C.item_ready[0], 0, abort_flag)) {   // K producer: Q of a first chain item
    const int e0 = C.item_e[0];
    if (e0 >= 0 && e0 < n_items) {
      const ItemView v0 = view(C.item[0]);
      if (v0.n_tiles > 0 && v0.kind == kItemChain) q_tma_start(v0, 0);
    }
  }

  for (;;) {
    const int slot = item_seq & 1;
    // the descriptor of this item was published during the previous one (or before the loop)
    bool have = mbar_wait(&C.item_ready[slot], (item_seq >> 1) & 1, abort_flag);
    const int e = have ? C.item_e[slot] : -1;
    if (e < 0 || e >= n_items) break;
    const ItemView it = view(C.item[slot]);
    const int n_tiles = it.n_tiles;
    if (tid == (kSoftmaxWarps + 3) * 32 + 1) fetch_item(slot ^ 1);   // a lane that has nothing else to do

    if (warp < kSoftmaxWarps) {
      // =================================================== softmax + epilogue ==================================
      // One thread per query row (= one TMEM lane), 128 score columns per tile.
      const int row = tid;
      const int i = row / G, hl = row - i * G;
      const bool row_valid = i < it.n_tok;
      const int h = it.g * G + hl;
      int64_t q_row = 0;                                          // output row
      int dec = 0;
      if (row_valid) {
        if (it.kind == kItemChain) q_row = it.tok0 + i;
        else { dec = it.tok0 + i; q_row = P.dec_tok[dec]; }
      }
      const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
      float m = -INFINITY, m_next = -INFINITY, l = 0.f;
      bool ok = true;
      if (n_tiles > 0) {
        int limit_row = (it.kind == kItemChain) ? it.limit0 + i : it.limit0;
        if (limit_row > it.kv_end) limit_row = it.kv_end;
        // first tile in which some row of this warp has a masked column (causal tail / end of the source): tiles
        // before it need neither the mask nor a vote about it
        const int first_masked_tile = __reduce_min_sync(0xffffffffu, max(limit_row - it.kv_begin, 0) / kTile);
        for (int j = 0; j < n_tiles; ++j) {
          const uint32_t gj = g_tile + j;
          const int b = gj % kRing;
          const uint32_t s_col = kColS + b * kTile;
          // (no vote and no early exit here: after a wait has run out the CTA is aborting, the later waits fail fast
          // and the thread runs the rest of the item on whatever it finds; `ok` keeps the result from being written)
          if (!mbar_wait(&C.s_full[b], (gj / kRing) & 1, abort_flag)) ok = false;
          tc_fence_after();
          // the second half of the scores is fetched while the exponentials of the first half are computed
          uint32_t sr[kTile];
          tmem_ld32(tmem + lane_base + s_col, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
          tmem_ld32(tmem + lane_base + s_col + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
          tmem_wait_ld();
          tmem_ld32(tmem + lane_base + s_col + 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
          tmem_ld32(tmem + lane_base + s_col + 96, *reinterpret_cast<uint32_t(*)[32]>(&sr[96]));

          const int pos0 = it.kv_begin + j * kTile;
          const bool masked = j >= first_masked_tile;             // warp-uniform
          if (masked) {                                           // causal tail or end of the source
            tmem_wait_ld();
            tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
            tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
            const int nvis = limit_row - pos0;                    // visible columns of this tile for this row
#pragma unroll
            for (int c = 0; c < kTile; ++c)
              if (c >= nvis) sr[c] = 0xff800000u;                 // -inf
          }
          // Reference maximum, one tile behind: the exponentials of this tile are taken relative to the reference m
          // that the previous tiles produced, so they do not have to wait for this tile's own maximum, which is
          // computed alongside them (the SFU pipe bounds the loop; the FMNMX are free) and only decides the
          // reference of the NEXT tile (when it exceeds m by more than 2^kLazyLog2, so O is rarely rescaled).
          // out = O / l and lse = m*scale + ln l hold for any m; only the fp32 range limits how far a score may
          // exceed the reference, hence the exact fallback below when a tile jumps by more than 2^kJumpLog2 (always
          // the case for the first visible key, where m = -inf).
          float alpha = 1.f;
          if (m_next != m) {                                      // decided by the previous tile
            alpha = ex2((m - m_next) * cl2);
            m = m_next;
            l *= alpha;
          }
          if (j == 0) {                                           // no reference yet: take this tile's exact maximum first
            tmem_wait_ld();                                       // (instead of exponentials that the fallback would redo)
            tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
            tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
            float e4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < kTile; c += 2)
              e4[(c >> 1) & 3] = max3(e4[(c >> 1) & 3], __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
            const float mxe = fmaxf(fmaxf(e4[0], e4[1]), fmaxf(e4[2], e4[3]));
            if (mxe > -INFINITY) { m = mxe; m_next = mxe; }
          }
          float mc = m == -INFINITY ? 0.f : m * cl2;
          // Every instruction of this loop costs an issue slot that the SFU does not hide (an ex2 holds the
          // sub-partition for 8 clocks and the rest adds to it), so the scaling and the row sum work on fp32 pairs.
          const f32x2 cl2_2 = pack2(cl2, cl2);
          f32x2 nmc2 = pack2(-mc, -mc);
          f32x2 sum2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          uint32_t pr[kTile / 2];
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) {
            if (hf == 1) {
              tmem_wait_ld();                                     // (no-op when the mask path has waited already)
              tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
              tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
            }
#pragma unroll
            for (int c = hf * 64; c < hf * 64 + 64; c += 2) {
              const float s0 = __uint_as_float(sr[c]), s1 = __uint_as_float(sr[c + 1]);
              float x0, x1;
              unpack2(fma2(pack2(s0, s1), cl2_2, nmc2), x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              sum2[(c >> 1) & 1] = add2(sum2[(c >> 1) & 1], pack2(p0, p1));
              pr[c >> 1] = pack_bf16_rn(p0, p1);
              if ((c & 6) == 0) mx4[(c >> 3) & 3] = max3(mx4[(c >> 3) & 3], s0, s1);   // every fourth pair
            }
          }
          float sum4[4];
          unpack2(sum2[0], sum4[0], sum4[1]);
          unpack2(sum2[1], sum4[2], sum4[3]);
          // mx: maximum of a sample of the columns (enough to move the reference lazily).  A score far above the
          // reference shows in the row sum of the tile instead, which costs nothing to test.
          float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          const float tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
          const bool jump = m == -INFINITY || !(tile_sum <= jump_sum);   // no reference yet, or beyond 2^kJumpLog2 / inf / NaN
          const int n_keys = min(kTile, it.kv_end - pos0);
          // one vote covers every rare path of a tile: exact fallback, O rescale, ragged end of the source
          const bool rare = __any_sync(0xffffffffu, jump || (alpha != 1.f && j > 0)) || n_keys < kTile;
          if (rare && __any_sync(0xffffffffu, jump)) {
            if (jump) {                                           // exact path: this tile's own maximum is the reference
#pragma unroll
              for (int c = 0; c < kTile; c += 2)
                mx4[(c >> 1) & 3] = max3(mx4[(c >> 1) & 3], __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
              mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            }
            if (jump && mx > -INFINITY) {
              const float a2 = ex2((m - mx) * cl2);               // 0 when the row had no visible key so far
              alpha *= a2;
              l *= a2;
              m = mx;
              mc = m * cl2;
              sum4[0] = sum4[1] = sum4[2] = sum4[3] = 0.f;
#pragma unroll
              for (int c = 0; c < kTile; c += 2) {
                const float p0 = ex2(__uint_as_float(sr[c]) * cl2 - mc);
                const float p1 = ex2(__uint_as_float(sr[c + 1]) * cl2 - mc);
                sum4[(c >> 1) & 3] += p0 + p1;
                pr[c >> 1] = pack_bf16_rn(p0, p1);
              }
            }
          }
          l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
          m_next = mx > m + lazy_raw ? mx : m;
          const bool move = alpha != 1.f;

          if (rare && __any_sync(0xffffffffu, move && j > 0)) {   // rescale O (warp-collective TMEM access)
            ok = mbar_wait(&C.pv_done[(gj - 1) % kRing], ((gj - 1) / kRing) & 1, abort_flag);   // PV(j-1) has landed in O
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
              uint32_t o0[32];
              tmem_ld32(tmem + lane_base + kColO + c0, o0);
              tmem_wait_ld();
#pragma unroll
              for (int x = 0; x < 32; ++x) o0[x] = __float_as_uint(__uint_as_float(o0[x]) * alpha);
              tmem_st32(tmem + lane_base + kColO + c0, o0);
            }
            tmem_wait_st();
          }
          // ---- last tile of a source that ends inside a page / inside the tile: zero the V rows past the end ---
          if (n_keys < kTile) {
            const int s = gj % kStagesV;
            ok = mbar_wait(&C.v_full[s], (gj / kStagesV) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            uint8_t* vs = smem + kOffV + s * kStageBytes;
            const int n_chunks = (kTile - n_keys) * 16;           // 16-byte chunks to clear (both halves)
            for (int x = tid; x < n_chunks; x += kSoftmaxWarps * 32) {
              const int r = n_keys + (x >> 4), cc = x & 15;
              *reinterpret_cast<uint4*>(vs + (cc >> 3) * (kStageBytes / 2) + r * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
          }
          // ---- P (bf16 pairs) over the first 64 columns of its own S buffer: the A operand of PV, read from TMEM ------
#pragma unroll
          for (int c0 = 0; c0 < kTile / 2; c0 += 32)
            tmem_st32(tmem + lane_base + s_col + c0, *reinterpret_cast<uint32_t(*)[32]>(&pr[c0]));
          tmem_wait_st();
          if (n_keys < kTile) fence_proxy_async_smem();           // the V rows cleared above
          tc_fence_before();
          mbar_arrive(&C.p_full[b]);
        }
        ok = __all_sync(0xffffffffu, ok);
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
          if (!row_valid) continue;
          if (final_out) {
            __nv_bfloat16* dst = P.out + (q_row * P.Hq + h) * kHeadDim + c0;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              uint32_t w[8];
#pragma unroll
              for (int y = 0; y < 8; ++y)
                w[y] = pack_bf16_rn(__uint_as_float(orow[16 * x + 2 * y]) * inv, __uint_as_float(orow[16 * x + 2 * y + 1]) * inv);
              st_global_32B(dst + 16 * x, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          } else {
            float* dst = P.part_o + (slot * P.Hq + h) * kHeadDim + c0;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              uint32_t w[8];
#pragma unroll
              for (int y = 0; y < 8; ++y) w[y] = __float_as_uint(__uint_as_float(orow[8 * x + y]) * inv);
              st_global_32B(dst + 8 * x, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          }
        }
        if (row_valid) {
          if (final_out) { if (P.lse) P.lse[q_row * P.Hq + h] = lse; }
          else P.part_lse[slot * P.Hq + h] = lse;
        }
      }
    } else if (warp < kSoftmaxWarps + 2) {
      // =================================================== TMA producers ========================================
      // Warp kSoftmaxWarps streams the K tiles, the next warp the V tiles, each as far ahead of its own consumer as
      // its ring allows.  After the last tile of this item the warp goes on with the first tiles of the NEXT item
      // (whose descriptor a spare lane has fetched meanwhile): their stages become free as this item's products
      // complete, so the next item's first tiles are in shared memory by the time this item has drained.
      const int which = warp - kSoftmaxWarps;                    // 0: K, 1: V
      const int n_stages = which ? kStagesV : kStagesK;
      const CUtensorMap* tm = which ? &tmap_v : &tmap_k;
      uint64_t* full = which ? C.v_full : C.k_full;
      uint64_t* empty = which ? C.v_empty : C.k_empty;
      uint8_t* ring = smem + (which ? kOffV : kOffK);
      int* seg_first = C.seg_first_page[which];
      long long* seg_off = C.seg_page_off[which];
      // tiles [j_begin, j_end) of item `v`; calls follow one another in tile order, so the stage counters run on
      auto stream_tiles = [&](const ItemView& v, int j_begin, int j_end) -> bool {
        if (j_begin >= j_end) return true;
        if (lane == 0) {
          int n_seg = 0;
          if (v.kind == kItemChain) {
            int chain[SS_MAX_DEPTH];
            int d = 0;
            for (int a = v.node; a >= 0 && d < SS_MAX_DEPTH; a = P.node_parent[a]) chain[d++] = a;
            int first = 0;
            for (int c = d - 1; c >= 0; --c) {
              const int n = chain[c];
              const int np = (P.node_kv_len[n] + kPage - 1) / kPage;
              if (np == 0) continue;
              seg_first[n_seg] = first;
              seg_off[n_seg] = P.node_page_offsets[n];
              first += np;
              ++n_seg;
            }
            seg_first[n_seg] = first;
          } else {
            seg_first[0] = 0;
            seg_off[0] = P.node_page_offsets[v.node];
            seg_first[1] = 0x7fffffff;
            n_seg = 1;
          }
          C.n_seg[which] = n_seg;
        }
        __syncwarp();
        const int n_seg = C.n_seg[which];
        // row coordinate (in the pool viewed as rows of 128 elements) of page `pg` of tile j's (page, kv head) block
        auto page_coord = [&](int j, int pg) -> int {
          if (j >= j_end) return 0;
          const int pos0 = v.kv_begin + j * kTile;
          const int n_pages = (min(kTile, v.kv_end - pos0) + kPage - 1) / kPage;
          if (pg >= n_pages) return 0;
          const int vp = pos0 / kPage + pg;
          int d = 0;
          while (d + 1 < n_seg && vp >= seg_first[d + 1]) ++d;
          const int64_t phys = P.node_pages[seg_off[d] + (vp - seg_first[d])];
          return static_cast<int>((phys * P.page_stride + static_cast<int64_t>(v.g) * P.head_stride) >> 7);
        };
        bool ok = true;
        // The page ids of four tiles are fetched with one load per lane (lane = 8 * tile-in-block + page), a whole
        // block ahead of their use: the dependent global load is off the per-tile path.  The lanes hand them to ONE
        // elected lane through shared memory, and that lane issues all copies of the block in straight-line code:
        // bulk-tensor copies are issued from uniform registers, and under a branch that several lanes may take the
        // compiler wraps each of them in a loop over the active lanes (about a dozen instructions per copy, all of
        // them issue slots taken from the softmax warp of the same sub-partition).
        int* coords = C.page_coord[which];
        int cur = page_coord(j_begin + (lane >> 3), lane & 7);
        for (int j0 = j_begin; j0 < j_end && ok; j0 += 4) {
          const int nxt = page_coord(j0 + 4 + (lane >> 3), lane & 7);
          const int n_blk = min(4, j_end - j0);
          coords[lane] = cur;
          __syncwarp();
          if (elect_one()) {
            int s = prod_stage;
            uint32_t u = prod_wraps;
            for (int t = 0; t < n_blk; ++t) {
              const int pos0 = v.kv_begin + (j0 + t) * kTile;
              const int n_pages = (min(kTile, v.kv_end - pos0) + kPage - 1) / kPage;
              if (u > 0 && !mbar_wait(&empty[s], (u - 1) & 1, abort_flag)) { ok = false; break; }
              mbar_arrive_expect_tx(&full[s], static_cast<uint32_t>(n_pages) * 4096u);
              const int4 y03 = *reinterpret_cast<const int4*>(&coords[t * 8]);
              const int4 y47 = *reinterpret_cast<const int4*>(&coords[t * 8 + 4]);
              const int y[8] = {y03.x, y03.y, y03.z, y03.w, y47.x, y47.y, y47.z, y47.w};
              uint8_t* dst = ring + s * kStageBytes;
#pragma unroll
              for (int pg = 0; pg < kTile / kPage; ++pg) {
                if (pg < n_pages) {
                  tma_load_2d(dst + pg * 2048, tm, 0, y[pg], &full[s]);
                  tma_load_2d(dst + kStageBytes / 2 + pg * 2048, tm, 64, y[pg], &full[s]);
                }
              }
              if (++s == n_stages) { s = 0; ++u; }
            }
          }
          __syncwarp();                                          // the elected lane has read the coordinates
          ok = __all_sync(0xffffffffu, ok);
          prod_stage += n_blk;                                   // every lane keeps the counters
          while (prod_stage >= n_stages) { prod_stage -= n_stages; ++prod_wraps; }
          cur = nxt;
        }
        __syncwarp();                                            // the segment tables are rewritten by the next call
        return ok;
      };
      if (which == 1 && q_pending) {                               // the Q rows gathered during the previous item
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&C.q_full);
        q_pending = false;
      }
      bool ok = stream_tiles(it, n_prefetched, n_tiles);
      n_prefetched = 0;
      // ---- the first tiles of the next item --------------------------------------------------------------------
      if (ok) ok = mbar_wait(&C.item_ready[slot ^ 1], ((item_seq + 1) >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        const int e_next = C.item_e[slot ^ 1];
        if (e_next >= 0 && e_next < n_items) {
          const ItemView nv = view(C.item[slot ^ 1]);
          n_prefetched = min(nv.n_tiles, n_stages);
          // Q buffer slot ^ 1 is free: the products of the item before this one have completed
          if (which == 0 && nv.n_tiles > 0 && nv.kind == kItemChain && elect_one()) q_tma_start(nv, slot ^ 1);
          // Q buffer slot ^ 1 is free: the products of the item before this one have completed
          if (which == 1 && nv.n_tiles > 0 && nv.kind != kItemChain) { q_gather_start(nv, slot ^ 1); q_pending = true; }
          if (!stream_tiles(nv, 0, n_prefetched)) n_prefetched = 0;   // (aborting)
        }
      }
    } else if (warp == kSoftmaxWarps + 2) {
      // =================================================== S = Q K^T issuer ====================================
      if (n_tiles > 0 && elect_one()) {                          // (elected, not `lane == 0`: see the producers)
        constexpr uint32_t idesc_qk = instr_desc_bf16(128, kTile, false);
        const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + kOffQ + slot * 32768), 0, 1024);
        const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + kOffK), 0, 1024);
        bool ok = it.kind == kItemChain ? mbar_wait(&C.q_full_tma, q_uses_tma & 1, abort_flag)
                                        : mbar_wait(&C.q_full, (q_uses - q_uses_tma) & 1, abort_flag);
        for (int j = 0; j < n_tiles && ok; ++j) {
          const uint32_t gj = g_tile + j;
          const int s = gj % kStagesK, b = gj % kRing;
          // buffer b held S / P of tile j - kRing: free once the P V product that read it has completed
          if (j >= kRing) ok = mbar_wait(&C.pv_done[b], ((gj - kRing) / kRing) & 1, abort_flag);
          ok = ok && mbar_wait(&C.k_full[s], (gj / kStagesK) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t k_desc = smem_desc_advance(k_desc0, static_cast<uint32_t>(s) * kStageBytes);
          const uint32_t d_tmem = tmem + kColS + b * kTile;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_bf16_ss(d_tmem, smem_desc_advance(q_desc0, (kk >> 2) * 16384 + (kk & 3) * 32),
                        smem_desc_advance(k_desc, (kk >> 2) * (kStageBytes / 2) + (kk & 3) * 32), idesc_qk,
                        kk > 0 ? 1u : 0u);
          mma_commit(&C.k_empty[s]);
          mma_commit(&C.s_full[b]);
        }
      }
    } else {
      // =================================================== O += P V issuer =====================================
      if (n_tiles > 0 && elect_one()) {
        constexpr uint32_t idesc_pv = instr_desc_bf16(128, kHeadDim, true);
        const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + kOffV), kStageBytes / 2, 1024);
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
          const uint32_t gj = g_tile + j;
          const int s = gj % kStagesV, b = gj % kRing;
          ok = mbar_wait(&C.v_full[s], (gj / kStagesV) & 1, abort_flag) &&
               mbar_wait(&C.p_full[b], (gj / kRing) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t v_desc = smem_desc_advance(v_desc0, static_cast<uint32_t>(s) * kStageBytes);
          const uint32_t o_tmem = tmem + kColO, p_tmem = tmem + kColS + b * kTile;
#pragma unroll
          for (int kk = 0; kk < kTile / 16; ++kk)
            mma_bf16_ts(o_tmem, p_tmem + kk * 8, smem_desc_advance(v_desc, kk * 2048), idesc_pv,
                        (j > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&C.v_empty[s]);
          mma_commit(&C.pv_done[b]);
          if (j + 1 == n_tiles) mma_commit(&C.o_final);
        }
      }
    }
    // ---- item end: every role meets here, so the next item starts from a drained pipeline --------------------
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    g_tile += n_tiles;
    if (n_tiles > 0) {
      ++q_uses;
      if (it.kind == kItemChain) ++q_uses_tma;
    }
    ++item_seq;
  }

  // ---- teardown --------------------------------------------------------------------------------------------------
  __syncthreads();
  if (C.abort_flag) {
    if (tid == 0) set_status(&P.hdr->status, SS_ERR_TIMEOUT);
    const long long t0 = clock64();                 // let copies / MMAs that are still in flight land
    while (clock64() - t0 < 4000000LL) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == kSoftmaxWarps) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace deep

int32_t launch_tile_items_umma_deep(const Params& P, cudaStream_t st, int sm_count) {
  using namespace deep;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(tile_items_umma_deep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    configured = true;
  }
  const int64_t rows = ((P.num_pages > 0 ? P.num_pages - 1 : 0) * P.page_stride + (P.Hkv - 1) * P.head_stride) / 128 + kPage;
  if (rows >= 0x7fffffffLL) return SS_ERR_UNSUPPORTED;
  CUtensorMap tk, tv;
  if (!tmap::encode_2d_bf16(&tk, P.k_pool, kHeadDim, static_cast<uint64_t>(rows), kHeadDim * 2, kPage) ||
      !tmap::encode_2d_bf16(&tv, P.v_pool, kHeadDim, static_cast<uint64_t>(rows), kHeadDim * 2, kPage))
    return SS_ERR_CUDA;
  // one CTA per SM: the kernel takes all 512 TMEM columns and most of the shared memory
  CUtensorMap tq;
  const int64_t q_rows = P.q_src_offsets ? P.q_src_rows : P.total_q;
  if (!tmap::encode_q_bf16(&tq, P.q, static_cast<uint64_t>(P.Hq), static_cast<uint64_t>(q_rows > 0 ? q_rows : 1),
                           static_cast<uint32_t>(P.G), static_cast<uint32_t>(P.tok_per_tile)))
    return SS_ERR_CUDA;
  SS_LAUNCH(tile_items_umma_deep_kernel, sm_count, kUmmaThreads, kUmmaSmem, st, tk, tv, tq, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
