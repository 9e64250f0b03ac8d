// Tensor-core tile kernel of ss_tree_attention (tcgen05 + TMEM + TMA), the default: one CTA per SM that owns all 512
// TMEM columns and works on 128-key tiles.  Same items and the same arithmetic as the two-CTAs-per-SM kernel in
// attn_umma.cu (a 64-key tile there); what differs follows from measurements on this part:
//   * an SM retires one tcgen05 instruction (MMA or commit) per ~50 clocks whatever its shape, and a 64-key tile costs
//     17 of them: with 128-key tiles every MMA is M128 x N128 x K16 (64 clocks of math) and the count per key halves;
//   * an ex2 occupies the special-function unit of an SM sub-partition for 8 clocks, and in the dependent chain of the
//     softmax loop (scale, exponential, sum, convert; 168 registers leave little room to interleave pairs) nearly
//     every other instruction adds to that, so the loop works on packed fp32 pairs, takes the row maximum from a
//     sample of the columns inside the exponential loop, and uses a reference maximum that lags one tile behind;
//   * a score buffer is recycled only when the P V product that read it has completed, so with two buffers the chain
//     Q K^T -> softmax -> P V of one tile bounds the next but one: three S/P buffers (128 columns each) + O (128
//     columns) fill the TMEM exactly, Q stays in shared memory;
//   * with one softmax thread per row that thread needs all 254 registers and spends a third of each tile in exposed
//     latencies.  Here TWO threads share a row: the two warps that can reach a TMEM lane quarter (w and w + 4) each
//     take 64 of the row's 128 scores, so a thread holds 64 scores + 32 packed P values (168 registers are plenty)
//     and each sub-partition has two softmax warps to interleave.
// What the two threads of a row must agree on is the reference maximum.  For the first tile of an item they exchange
// the exact maxima of their halves (a 64-thread barrier, once per item); from then on each posts the sampled maximum
// of its half to a shared-memory mailbox after every tile and reads the other's post of the PREVIOUS tile, so both
// compute the same lagged reference without waiting for each other.  P of the two halves goes over the first 32
// columns of each thread's own 64 score columns (columns 0..31 and 64..95 of the S buffer).  Row sums are kept per
// half and added in the epilogue (second 64-thread barrier), where each half also writes 64 output columns.  A half
// row whose exponentials leave the range of the lagged reference (scores rising by more than 2^40 from one tile to
// the next) cannot be repaired in place, because the other half has used the same reference: it marks the item, and
// when the item's tiles are through, all warps of the CTA recompute it exactly on the CUDA cores (attn_rows.cuh).
// Roles: warps 0-7 softmax + epilogue; warp 8 streams K tiles and warp 9 V tiles through TMA (3 and 2 stages of
// 32 KB); an elected lane of warp 10 issues S[b] = Q K^T (8 MMAs per tile), of warp 11 O += P[b] V (8 MMAs, P read
// from TMEM, V MN-major); lane 1 of warp 11 fetches the NEXT item while this one runs: the producers then load its
// first K / V tiles and its Q rows (a 3-D TMA box for a chain item, issued by the K producer; cp.async of the
// gathered rows of a stacked item by the V producer warp) into the second Q buffer before the current item has
// drained, and the Q K^T issuer goes on with the next item's first two products as soon as it has issued the current
// item's last.  The softmax warps do nothing but the softmax and the epilogue.
// Every wait is bounded; on expiry the CTA raises its abort flag, the later waits fail fast, the roles run through
// the item's remaining tiles without writing results, the CTA frees its TMEM and the kernel records SS_ERR_TIMEOUT.
#include "attn_plan.cuh"
#include "attn_rows.cuh"
#include "umma.cuh"

namespace ss {
namespace attn {

using namespace umma;

namespace split {

constexpr int kSoftmaxWarps = 8;               // two warps per TMEM lane quarter: each takes 64 of a row's 128 scores
constexpr int kUmmaThreads = (kSoftmaxWarps + 4) * 32;
constexpr int kTile = 128;                     // keys per tile (two of the planner's 64-key tiles)
constexpr int kStageBytes = kTile * 256;       // one K or V tile: [16 groups of 8 keys][2 halves of 64 dims][8 rows][128 B]
constexpr int kStagesK = 3;
constexpr int kStagesV = 2;                    // V is consumed a softmax later than K: two stages are enough
constexpr int kRing = 3;                       // S/P buffers
#ifndef SS_PRE_ISSUE
#define SS_PRE_ISSUE 2
#endif
constexpr int kPreIssue = SS_PRE_ISSUE;        // Q K^T products of the next item issued before the current one ends (< kRing)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                  // kRing x kTile columns
constexpr uint32_t kColO = kRing * kTile;      // 128 columns
constexpr float kLazyLog2 = 8.0f;              // the reference maximum moves only when exceeded by 2^8
constexpr float kJumpLog2 = 40.0f;             // exponentials may exceed the reference by at most 2^40 (+2^8 lag)
constexpr int kOffQ = 0;                       // 2 buffers (this item / next item) x [2 halves of 64 dims][128 rows][128 B]
constexpr int kOffK = 65536;
constexpr int kOffV = kOffK + kStagesK * kStageBytes;
constexpr int kUmmaSmem = kOffV + kStagesV * kStageBytes;   // + the control block in static shared memory
static_assert(kColO + kHeadDim <= kTmemCols && kColS + kRing * kTile <= kColO, "score buffers and accumulator inside the allocated TMEM columns");

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
  // Sampled tile maxima of the two halves of a row, one tile behind: [tile parity][half][row], the low two bits of the
  // value replaced by a tag (1 or 2) that tells the reader which tile the value belongs to.  The two exchanges per
  // item that go through a pair barrier (exact maximum of the first tile, row sums at the end) borrow the slot that
  // is idle at that moment and leave it cleared (tag 0 matches nothing).
  uint32_t xmax[2][2][128];
  int overflow[2];                               // (per item slot) a half-row left the range of the lagged reference:
                                                 // the item is computed again, exactly, when its tiles are through
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

__device__ __forceinline__ uint32_t ld_shared_volatile(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_shared(uint32_t addr, uint32_t v) {
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
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

// Out of line on purpose: code that is inlined into the kernel costs its hot loops registers and instruction-cache
// space even when it never runs.
__device__ __noinline__ void exact_second_pass(const Params& P, const TileItem* it, int warp, int lane) {
  tile_item_rows_exact(P, *it, warp, kUmmaThreads / 32, lane);
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
tile_items_umma_split_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                            const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ Params P) {
  // The block first sets up what needs nothing from the kernels before it (barriers, the zeroed Q buffers, tensor
  // memory): launched with programmatic serialization it may be resident while the planner is still running, and
  // this part then overlaps the planner's tail.  It waits for the planner right after (see below).
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
  for (int x = tid; x < 2 * 2 * 128; x += kUmmaThreads) (&C.xmax[0][0][0])[x] = 0u;   // tag 0: nothing posted
  if (tid == 0) C.overflow[0] = C.overflow[1] = 0;
  fence_proxy_async_smem();
  if (warp == kSoftmaxWarps) tmem_alloc(&C.tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // ---- from here on the planner's results are read: wait for it, then let the leaf kernel behind this one start
  //      (it needs the plan too, and nothing from this kernel until it merges)
  ss::grid_dependency_enter_then_release();
  SS_STAMP_BEGIN(P.hdr, 2);
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
  auto fetch_item = [&](int dst, bool first_fetch) {
    // (a block's first item is its own index: no trip to the counter before the first tile; the counter hands out
    //  the items after the first gridDim.x)
    int e = -1;
    if (P.hdr->status == SS_OK && !C.abort_flag)
      e = first_fetch ? static_cast<int>(blockIdx.x) : atomicAdd(&P.hdr->tile_counter, 1) + static_cast<int>(gridDim.x);
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
      SS_CHECK_OR(q_src >= 0 && q_src < (P.q_src_offsets ? P.q_src_rows : P.total_q), &P.hdr->status, q_src = 0);
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

  if (tid == 0) fetch_item(0, true);
  __syncthreads();
  bool q_pending = false;   // V producer warp: the gather of the first item's Q rows is under way
  int qk_pre = 0;           // Q K^T issuer warp: products of the coming item that were issued during the one before
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

#ifdef SS_STAMPS
  long long tl_wait = 0, tl_ld = 0, tl_ref = 0, tl_exp = 0, tl_store = 0, tl_mark = 0, tl_tiles = 0;
  long long acc_first_s = 0, acc_tiles = 0, acc_o_wait = 0, acc_epi = 0, acc_sync = 0, acc_items = 0, t_mark = 0;
#endif
  for (;;) {
    const int slot = item_seq & 1;
#ifdef SS_STAMPS
    if (tid == 0) t_mark = clock64();
#endif
    // the descriptor of this item was published during the previous one (or before the loop)
    bool have = mbar_wait(&C.item_ready[slot], (item_seq >> 1) & 1, abort_flag);
    const int e = have ? C.item_e[slot] : -1;
    if (e < 0 || e >= n_items) break;
    const ItemView it = view(C.item[slot]);
    const int n_tiles = it.n_tiles;
    if (tid == (kSoftmaxWarps + 3) * 32 + 1) fetch_item(slot ^ 1, false);   // a lane that has nothing else to do

    if (warp < kSoftmaxWarps) {
      // =================================================== softmax + epilogue ==================================
      // Two threads per query row (= TMEM lane): thread `hf` of the pair takes score columns [64 hf, 64 hf + 64) of
      // every tile, keeps its own partial row sum and writes output columns [64 hf, 64 hf + 64).  Both derive the
      // same reference maximum: from the exact half maxima of the first tile (exchanged through a pair barrier) and,
      // one tile behind, from the sampled maxima that each posts for the other.
      const int hf = warp >> 2;
      const int row = tid & 127;
      const int i = row / G, hl = row - i * G;
      const bool row_valid = i < it.n_tok;
      const int h = it.g * G + hl;
      // where the row goes: the output row of a chain item's token, the partial slot of a stacked item's token (read
      // now, so that the load is long done when the epilogue needs it)
      int64_t out_row = 0;
      if (row_valid) out_row = it.kind == kItemChain ? static_cast<int64_t>(it.tok0 + i)
                                                     : static_cast<int64_t>(P.dec_slot_base[it.tok0 + i]) + it.slot_off;
      const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
      auto pair_barrier = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(2 + (warp & 3)) : "memory"); };
      float m = 0.f, l = 0.f;                                     // reference maximum (0 while the row has no visible key)
      uint32_t own_post = 0;                                      // what this thread posted for the previous tile
      bool ok = true;
      if (n_tiles > 0) {
        int limit_row = (it.kind == kItemChain) ? it.limit0 + i : it.limit0;
        if (limit_row > it.kv_end) limit_row = it.kv_end;
        const int first_masked_tile = __reduce_min_sync(0xffffffffu, max(limit_row - it.kv_begin, 0) / kTile);
        const int ragged_tile = ((it.kv_end - it.kv_begin) % kTile) ? n_tiles - 1 : -1;   // only a last tile can end early
        // Everything that depends on the tile number is carried along instead of recomputed (the two warps of a
        // sub-partition share its issue slots with each other and with a producer or MMA warp: instructions count).
        int b = g_tile % kRing;                                   // S buffer of the tile
        uint32_t b_phase = (g_tile / kRing) & 1;
        uint32_t par = g_tile & 1;                                // mailbox slot of the tile's post
        uint32_t tag = ((g_tile >> 1) & 1u) + 1u;                 // tag of the tile's post
        uint32_t tag_prev = (((g_tile - 1) >> 1) & 1u) + 1u;      // tag of the previous tile's post (slot par ^ 1)
        const uint32_t xm_own = smem_u32(&C.xmax[0][hf][row]), xm_oth = smem_u32(&C.xmax[0][hf ^ 1][row]);
        for (int j = 0; j < n_tiles; ++j) {
          const uint32_t gj = g_tile + j;
          const uint32_t s_col = kColS + b * kTile + hf * 64;     // this thread's 64 scores; its P goes over the first 32
#ifdef SS_STAMPS
          if (tid == 0) tl_mark = clock64();
#endif
          if (!mbar_wait(&C.s_full[b], b_phase, abort_flag)) ok = false;
#ifdef SS_STAMPS
          if (tid == 0 && j > 0) { const long long t = clock64(); tl_wait += t - tl_mark; tl_mark = t; }
#endif
#ifdef SS_STAMPS
          if (tid == 0 && j == 0) { const long long t = clock64(); acc_first_s += t - t_mark; t_mark = t; }
#endif
          tc_fence_after();
          uint32_t sr[64];
          tmem_ld32(tmem + lane_base + s_col, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
          tmem_wait_ld();
#ifdef SS_STAMPS
          if (tid == 0 && j > 0) { const long long t = clock64(); tl_ld += t - tl_mark; tl_mark = t; }
#endif
          tmem_ld32(tmem + lane_base + s_col + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));

          const bool masked = j >= first_masked_tile;             // warp-uniform
          bool second_in = false;
          if (masked || j == 0) {
            tmem_wait_ld();
            tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
            second_in = true;
            if (masked) {
              const int nvis = limit_row - (it.kv_begin + j * kTile + hf * 64);   // visible ones of this thread's columns
#pragma unroll
              for (int c = 0; c < 64; ++c)
                if (c >= nvis) sr[c] = 0xff800000u;               // -inf
            }
          }
          // ---- reference of this tile --------------------------------------------------------------------------------
          float alpha = 1.f;
          if (j == 0) {                                           // exact maximum of the first tile, both halves
            float e4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 64; c += 2)
              e4[(c >> 1) & 3] = max3(e4[(c >> 1) & 3], __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
            const float mine = fmaxf(fmaxf(e4[0], e4[1]), fmaxf(e4[2], e4[3]));
            uint32_t (*xch)[128] = C.xmax[par ^ 1];               // idle until the post of tile gj + 1
            xch[hf][row] = __float_as_uint(mine);
            pair_barrier();
            const float mxe = fmaxf(mine, __uint_as_float(xch[hf ^ 1][row]));
            m = mxe > -INFINITY ? mxe : 0.f;
            pair_barrier();
            xch[hf][row] = 0u;
          } else {                                                // lagged: the sampled maxima of the previous tile
            const uint32_t src = xm_oth + (par ^ 1u) * (2 * 128 * 4);
            uint32_t other = ld_shared_volatile(src);
            if ((other & 3u) != tag_prev) {                       // the other half is still inside the previous tile
              const long long t0 = clock64();
              while (((other = ld_shared_volatile(src)) & 3u) != tag_prev) {
                if (*abort_flag || clock64() - t0 > kWaitCycles) { *abort_flag = 1; ok = false; break; }
              }
            }
            // (the tag bits stay in: both threads of the row compare the same two words)
            const float mx_prev = fmaxf(__uint_as_float(own_post), __uint_as_float(other));
            if (mx_prev > m + lazy_raw) {
              alpha = ex2((m - mx_prev) * cl2);
              m = mx_prev;
              l *= alpha;
            }
          }
#ifdef SS_STAMPS
          if (tid == 0 && j > 0) { const long long t = clock64(); tl_ref += t - tl_mark; tl_mark = t; }
#endif
          const float mc = m * cl2;
          const f32x2 cl2_2 = pack2(cl2, cl2);
          const f32x2 nmc2 = pack2(-mc, -mc);
          f32x2 sum2[2] = {pack2(0.f, 0.f), pack2(0.f, 0.f)};
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          uint32_t pr[32];
#pragma unroll
          for (int part = 0; part < 2; ++part) {
            if (part == 1 && !second_in) {
              tmem_wait_ld();
              tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
            }
#pragma unroll
            for (int c = part * 32; c < part * 32 + 32; c += 2) {
              const float s0 = __uint_as_float(sr[c]), s1 = __uint_as_float(sr[c + 1]);
              float x0, x1;
              unpack2(fma2(pack2(s0, s1), cl2_2, nmc2), x0, x1);
              const float p0 = ex2(x0), p1 = ex2(x1);
              sum2[(c >> 1) & 1] = add2(sum2[(c >> 1) & 1], pack2(p0, p1));
              pr[c >> 1] = pack_bf16_rn(p0, p1);
              if ((c & 14) == 0) mx4[(c >> 4) & 3] = max3(mx4[(c >> 4) & 3], s0, s1);   // every eighth pair
            }
          }
#ifdef SS_STAMPS
          if (tid == 0 && j > 0) { const long long t = clock64(); tl_exp += t - tl_mark; tl_mark = t; }
#endif
          float sum4[4];
          unpack2(sum2[0], sum4[0], sum4[1]);
          unpack2(sum2[1], sum4[2], sum4[3]);
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          const float tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
          // post this tile's sampled maximum for the other half (finite or -inf; the tag marks the tile)
          own_post = (__float_as_uint(mx) & ~3u) | tag;
          st_shared(xm_own + par * (2 * 128 * 4), own_post);
          if (!(tile_sum <= jump_sum)) C.overflow[slot] = 1;     // beyond the lagged reference's range: exact pass needed
          l += tile_sum;
          const bool ragged = j == ragged_tile;
          // (only the first half's warps vote: they own O and the V tail, and a vote per tile in every warp costs 3 %)
          const bool rare = hf == 0 && (__any_sync(0xffffffffu, alpha != 1.f && j > 0) || ragged);
          if (rare) {
            if (__any_sync(0xffffffffu, alpha != 1.f && j > 0)) { // rescale O (warp-collective TMEM access)
              ok = mbar_wait(&C.pv_done[(gj - 1) % kRing], ((gj - 1) / kRing) & 1, abort_flag) && ok;
              tc_fence_after();
#pragma unroll 1
              for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
                uint32_t o0[32];
                tmem_ld32(tmem + lane_base + kColO + c0, o0);
                tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 32; ++x) o0[x] = __float_as_uint(__uint_as_float(o0[x]) * alpha);
                tmem_st32(tmem + lane_base + kColO + c0, o0);
              }
            }
            if (ragged) {                                         // zero the V rows past the end of the source
              const int n_keys = it.kv_end - (it.kv_begin + j * kTile);
              const int s = gj % kStagesV;
              ok = mbar_wait(&C.v_full[s], (gj / kStagesV) & 1, abort_flag) && ok;
              uint8_t* vs = smem + kOffV + s * kStageBytes;
              const int n_chunks = (kTile - n_keys) * 16;         // 16-byte chunks to clear (both halves)
              for (int x = row; x < n_chunks; x += 128) {
                const int r = n_keys + (x >> 4), cc = x & 15;
                *reinterpret_cast<uint4*>(vs + (r >> 3) * 2048 + (cc >> 3) * 1024 + (r & 7) * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
              }
              fence_proxy_async_smem();
            }
          }
          // ---- P (bf16 pairs) over the first 32 of this thread's own 64 score columns -------------------------------
          tmem_st32(tmem + lane_base + s_col, pr);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&C.p_full[b]);
#ifdef SS_STAMPS
          if (tid == 0 && j > 0) { const long long t = clock64(); tl_store += t - tl_mark; ++tl_tiles; }
#endif
          if (++b == kRing) { b = 0; b_phase ^= 1u; }
          tag_prev = tag;
          if (par) tag ^= 3u;                                     // (the tag changes with every second tile: 1 <-> 2)
          par ^= 1u;
        }
        ok = __all_sync(0xffffffffu, ok);
#ifdef SS_STAMPS
        if (tid == 0) { const long long t = clock64(); acc_tiles += t - t_mark; t_mark = t; }
#endif
        if (ok) {
          ok = mbar_wait(&C.o_final, q_uses & 1, abort_flag);
          ok = __all_sync(0xffffffffu, ok);
          tc_fence_after();
        }
      }
#ifdef SS_STAMPS
      if (tid == 0) { const long long t = clock64(); acc_o_wait += t - t_mark; t_mark = t; }
#endif
      // ---- epilogue: the two halves add their row sums; each writes 64 output columns ---------------------------------
      C.xmax[0][hf][row] = __float_as_uint(l);                  // (every tile of the item is behind both halves here)
      pair_barrier();
      const float l_all = l + __uint_as_float(C.xmax[0][hf ^ 1][row]);
      pair_barrier();
      C.xmax[0][hf][row] = 0u;
#ifdef SS_CHECKED
      {                                                           // (warp-uniform outcome: the loads below are collective)
        const bool in_range = !row_valid || (out_row >= 0 && out_row < (it.slot_off < 0 ? P.total_q : static_cast<int64_t>(P.caps.slots)));
        if (!in_range) set_status(&P.hdr->status, SS_ERR_BAD_INPUT);
        if (!__all_sync(0xffffffffu, in_range)) ok = false;
      }
#endif
      if (ok) {
        const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
        const float lse = l_all > 0.f ? m * P.scale + __logf(l_all) : -INFINITY;
        const bool final_out = it.slot_off < 0;
#pragma unroll
        for (int c0 = hf * 64; c0 < hf * 64 + 64; c0 += 32) {
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
            __nv_bfloat16* dst = P.out + (out_row * P.Hq + h) * kHeadDim + c0;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
              uint32_t w[8];
#pragma unroll
              for (int y = 0; y < 8; ++y)
                w[y] = pack_bf16_rn(__uint_as_float(orow[16 * x + 2 * y]) * inv, __uint_as_float(orow[16 * x + 2 * y + 1]) * inv);
              st_global_32B(dst + 16 * x, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          } else {
            float* dst = P.part_o + (out_row * P.Hq + h) * kHeadDim + c0;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              uint32_t w[8];
#pragma unroll
              for (int y = 0; y < 8; ++y) w[y] = __float_as_uint(__uint_as_float(orow[8 * x + y]) * inv);
              st_global_32B(dst + 8 * x, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          }
        }
        if (row_valid && hf == 0) {
          if (final_out) { if (P.lse) P.lse[out_row * P.Hq + h] = lse; }
          else P.part_lse[out_row * P.Hq + h] = lse;
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
          int64_t phys = P.node_pages[seg_off[d] + (vp - seg_first[d])];
          SS_CHECK_OR(phys >= 0 && phys < P.num_pages, &P.hdr->status, phys = 0);
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
                  tma_load_4d(dst + pg * 4096, tm, 0, 0, 0, y[pg] >> 3, &full[s]);   // the whole (page, head) block
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
          const bool gather = which == 1 && nv.n_tiles > 0 && nv.kind != kItemChain;
          if (gather) q_gather_start(nv, slot ^ 1);
          if (!stream_tiles(nv, 0, n_prefetched)) n_prefetched = 0;   // (aborting)
          if (gather) {                        // published now: the Q K^T issuer starts on the next item before this one ends
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&C.q_full);
          }
        }
      }
    } else if (warp == kSoftmaxWarps + 2) {
      // =================================================== S = Q K^T issuer ====================================
      // After the products of this item the warp goes straight on with the first kPreIssue products of the NEXT item
      // (its Q rows and first K tiles were requested during this item): they run on the tensor pipe while the softmax
      // warps finish this item and write its rows out, and the next item finds its first scores waiting.
      int pre_next = 0;
      if (elect_one()) {                                         // (elected, not `lane == 0`: see the producers)
        constexpr uint32_t idesc_qk = instr_desc_bf16(128, kTile, false);
        const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + kOffK), 0, 2048);   // 8-key groups 2048 B apart
        // product of global tile gj with the Q rows in buffer `qbuf`; S buffer gj % kRing held S / P of tile
        // gj - kRing and is free once the P V product that read it has completed
        auto issue_qk = [&](uint32_t gj, int qbuf) -> bool {
          const int s = gj % kStagesK, b = gj % kRing;
          bool ok = gj < static_cast<uint32_t>(kRing) || mbar_wait(&C.pv_done[b], ((gj - kRing) / kRing) & 1, abort_flag);
          ok = ok && mbar_wait(&C.k_full[s], (gj / kStagesK) & 1, abort_flag);
          if (!ok) return false;
          tc_fence_after();
          const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + kOffQ + qbuf * 32768), 0, 1024);
          const uint64_t k_desc = smem_desc_advance(k_desc0, static_cast<uint32_t>(s) * kStageBytes);
          const uint32_t d_tmem = tmem + kColS + b * kTile;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_bf16_ss(d_tmem, smem_desc_advance(q_desc0, (kk >> 2) * 16384 + (kk & 3) * 32),
                        smem_desc_advance(k_desc, (kk >> 2) * 1024 + (kk & 3) * 32), idesc_qk,
                        kk > 0 ? 1u : 0u);
          mma_commit(&C.k_empty[s]);
          mma_commit(&C.s_full[b]);
          return true;
        };
        bool ok = true;
        if (n_tiles > qk_pre) {
          ok = it.kind == kItemChain ? mbar_wait(&C.q_full_tma, q_uses_tma & 1, abort_flag)
                                     : mbar_wait(&C.q_full, (q_uses - q_uses_tma) & 1, abort_flag);
          for (int j = qk_pre; j < n_tiles && ok; ++j) ok = issue_qk(g_tile + j, slot);
        }
        if (ok && mbar_wait(&C.item_ready[slot ^ 1], ((item_seq + 1) >> 1) & 1, abort_flag)) {
          const int e_next = C.item_e[slot ^ 1];
          if (e_next >= 0 && e_next < n_items) {
            const ItemView nv = view(C.item[slot ^ 1]);
            if (nv.n_tiles > 0) {
              const uint32_t used = n_tiles > 0 ? 1u : 0u;
              const uint32_t qn = q_uses + used, qn_tma = q_uses_tma + ((used && it.kind == kItemChain) ? 1u : 0u);
              ok = nv.kind == kItemChain ? mbar_wait(&C.q_full_tma, qn_tma & 1, abort_flag)
                                         : mbar_wait(&C.q_full, (qn - qn_tma) & 1, abort_flag);
              for (int j = 0; j < min(kPreIssue, nv.n_tiles) && ok; ++j) {
                ok = issue_qk(g_tile + n_tiles + j, slot ^ 1);
                if (ok) pre_next = j + 1;
              }
            }
          }
        }
      }
      qk_pre = __reduce_max_sync(0xffffffffu, pre_next);         // (the elected lane may differ from item to item)
    } else {
      // =================================================== O += P V issuer =====================================
      if (n_tiles > 0 && elect_one()) {
        constexpr uint32_t idesc_pv = instr_desc_bf16(128, kHeadDim, true);
        const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + kOffV), 1024, 2048);   // dims 64..127 1024 B on, 8-key groups 2048 B apart
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
          for (int kk = 0; kk < kTile / 16; ++kk)       // P of keys 0..63 at columns 0..31, of keys 64..127 at 64..95
            mma_bf16_ts(o_tmem, p_tmem + (kk >> 2) * 64 + (kk & 3) * 8, smem_desc_advance(v_desc, kk * 4096), idesc_pv,
                        (j > 0 || kk > 0) ? 1u : 0u);
          mma_commit(&C.v_empty[s]);
          mma_commit(&C.pv_done[b]);
          if (j + 1 == n_tiles) mma_commit(&C.o_final);
        }
      }
    }
#ifdef SS_STAMPS
    if (tid == 0) { const long long t = clock64(); acc_epi += t - t_mark; t_mark = t; }
#endif
    // ---- item end: every role meets here, so the next item starts from a drained pipeline --------------------
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
#ifdef SS_STAMPS
    if (tid == 0) { const long long t = clock64(); acc_sync += t - t_mark; ++acc_items; }
#endif
    // Exact second pass: the exponentials of some half-row overflowed the range of the lagged reference (scores that
    // rise by more than 2^40 from one tile to the next; the tensor-core pass has then written garbage for the
    // item).  All twelve warps recompute the item's rows on the CUDA cores, one row per warp and key by key.
    if (C.overflow[slot]) {
      exact_second_pass(P, &C.item[slot], warp, lane);
      __syncthreads();
      if (tid == 0) C.overflow[slot] = 0;
    }
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
  SS_STAMP_END(P.hdr, 3);
#ifdef SS_STAMPS
  if (tid == 0) {
    atomicAdd(&P.hdr->stamp[8], static_cast<unsigned long long>(acc_first_s));
    atomicAdd(&P.hdr->stamp[9], static_cast<unsigned long long>(acc_tiles));
    atomicAdd(&P.hdr->stamp[10], static_cast<unsigned long long>(acc_o_wait));
    atomicAdd(&P.hdr->stamp[11], static_cast<unsigned long long>(acc_epi));
    atomicAdd(&P.hdr->stamp[12], static_cast<unsigned long long>(acc_sync));
    atomicAdd(&P.hdr->stamp[13], static_cast<unsigned long long>(acc_items));
    atomicAdd(&P.hdr->stamp[14], static_cast<unsigned long long>(tl_wait));
    atomicAdd(&P.hdr->stamp[15], static_cast<unsigned long long>(tl_ld));
    atomicAdd(&P.hdr->stamp[16], static_cast<unsigned long long>(tl_ref));
    atomicAdd(&P.hdr->stamp[17], static_cast<unsigned long long>(tl_exp));
    atomicAdd(&P.hdr->stamp[18], static_cast<unsigned long long>(tl_store));
    atomicAdd(&P.hdr->stamp[19], static_cast<unsigned long long>(tl_tiles));
  }
#endif
}

}  // namespace split

int32_t launch_tile_items_umma(const Params& P, cudaStream_t st, int sm_count);   // the 64-key kernel (attn_umma.cu)

int32_t launch_tile_items_umma_split(const Params& P, cudaStream_t st, int sm_count) {
  using namespace split;
  // One bulk-tensor copy per (page, kv head) block needs the blocks to start on 8-row boundaries of the pool (rows of
  // 256 bytes); any other pool layout goes to the kernel that copies the two 64-dim halves of a block separately.
  if (P.page_stride % 1024 || P.head_stride % 1024) return launch_tile_items_umma(P, st, sm_count);
  static bool configured[kDeviceSlots] = {false};     // the attribute belongs to the (function, device) pair
  const int dev_slot = current_device_slot();
  if (dev_slot < 0 || !configured[dev_slot]) {
    if (cudaFuncSetAttribute(tile_items_umma_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    if (dev_slot >= 0) configured[dev_slot] = true;
  }
  const int64_t rows = ((P.num_pages > 0 ? P.num_pages - 1 : 0) * P.page_stride + (P.Hkv - 1) * P.head_stride) / 128 + kPage;
  if (rows >= 0x7fffffffLL) return SS_ERR_UNSUPPORTED;
  CUtensorMap tk, tv;
  if (!tmap::encode_kv_block_bf16(&tk, P.k_pool, static_cast<uint64_t>(rows)) ||
      !tmap::encode_kv_block_bf16(&tv, P.v_pool, static_cast<uint64_t>(rows)))
    return SS_ERR_CUDA;
  // one CTA per SM: the kernel takes all 512 TMEM columns and most of the shared memory
  CUtensorMap tq;
  const int64_t q_rows = P.q_src_offsets ? P.q_src_rows : P.total_q;
  if (!tmap::encode_q_bf16(&tq, P.q, static_cast<uint64_t>(P.Hq), static_cast<uint64_t>(q_rows > 0 ? q_rows : 1),
                           static_cast<uint32_t>(P.G), static_cast<uint32_t>(P.tok_per_tile)))
    return SS_ERR_CUDA;
  SS_LAUNCH(tile_items_umma_split_kernel, sm_count, kUmmaThreads, kUmmaSmem, st, tk, tv, tq, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
