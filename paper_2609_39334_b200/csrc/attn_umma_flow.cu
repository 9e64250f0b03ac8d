// Tensor-core tile kernel of ss_tree_attention (tcgen05 + TMEM + TMA), free-running version: the same tiles, the same
// softmax arithmetic and the same roles as the kernel in attn_umma_split.cu (one CTA per SM, 128-key tiles, two
// softmax threads per row, K and V streamed by two producer warps, one issuing thread for S = Q K^T and one for
// O += P V), but the roles no longer meet at the end of every item.  There an item costs about 8.5 k clocks on top of
// its tiles (drain of the last P V, epilogue, barrier, first Q K^T and first softmax of the next item with nothing
// else in flight) - a quarter of a 10-tile verification item.  Here:
//   * TMEM holds TWO score buffers (2 x 128 columns) and TWO output accumulators (2 x 128 columns): the P V products
//     of item k+1 accumulate into the other accumulator while item k's is being read out;
//   * the issuing threads and the producers run on into the next item as far as their rings allow (descriptors are
//     fetched two items ahead into a ring of 8 slots, Q is double-buffered and recycled through q_empty);
//   * the softmax warps do the first tile of item k+1 BEFORE the epilogue of item k: by then the last P V of item k has
//     long completed, and while they write item k's rows out the tensor pipe works on item k+1's second tile;
//   * an item whose exponentials left the range of the lagged reference is recomputed exactly by the eight softmax
//     warps at its (deferred) epilogue, the other roles keep going.
// Every wait is bounded; on expiry the CTA raises its abort flag, later waits fail fast, every role leaves its loop,
// the CTA frees its TMEM and the kernel records SS_ERR_TIMEOUT.
#include "attn_plan.cuh"
#include "attn_rows.cuh"
#include "umma.cuh"

namespace ss {
namespace attn {

using namespace umma;

namespace flow {

constexpr int kSoftmaxWarps = 8;               // two warps per TMEM lane quarter: each takes 64 of a row's 128 scores
constexpr int kUmmaThreads = (kSoftmaxWarps + 4) * 32;
constexpr int kTile = 128;                     // keys per tile
constexpr int kStageBytes = kTile * 256;       // one K or V tile: [16 groups of 8 keys][2 halves of 64 dims][8 rows][128 B]
constexpr int kStagesK = 3;
constexpr int kStagesV = 2;
constexpr int kRing = 2;                       // S/P buffers
constexpr int kItemRing = 8;                   // item descriptors in flight (the static shared memory has 3 KB in all)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                  // kRing x kTile columns
constexpr uint32_t kColO = kRing * kTile;      // 2 x 128 columns (items alternate)
constexpr float kLazyLog2 = 8.0f;              // the reference maximum moves only when exceeded by 2^8
constexpr float kJumpLog2 = 40.0f;             // exponentials may exceed the reference by at most 2^40 (+2^8 lag)
constexpr int kOffQ = 0;                       // 2 buffers x [2 halves of 64 dims][128 rows][128 B]
constexpr int kOffK = 65536;
constexpr int kOffV = kOffK + kStagesK * kStageBytes;
constexpr int kUmmaSmem = kOffV + kStagesV * kStageBytes;   // + the control block in static shared memory

struct Ctrl {
  // Ring barriers are indexed by a running count modulo the ring size and waited with the parity of (count / size); the
  // matching "free" barrier keeps a producer from running a whole ring ahead of its slowest consumer.
  uint64_t item_ready[kItemRing], item_free[kItemRing];        // descriptor slots (free: 8 softmax warps + 4 other roles)
  uint64_t q_full[2], q_empty[2];                              // Q buffers, by the count of items that have tiles
  uint64_t k_full[kStagesK], k_empty[kStagesK], v_full[kStagesV], v_empty[kStagesV];
  uint64_t s_full[kRing], p_full[kRing], pv_done[kRing];       // by global tile count
  uint64_t o_full[2], o_free[2];                               // accumulators, by the count of items that have tiles
  uint64_t pair_bar[4], epi_bar;                               // the two softmax warps of a lane quarter / all eight
  uint32_t tmem_slot;
  int abort_flag;
  int item_e[kItemRing];
  TileItem item[kItemRing];
  int overflow[kItemRing];                       // a half-row of the item left the range of the lagged reference
  // Sampled tile maxima of the two halves of a row, one tile behind: [tile parity][half][row]; the upper 16 bits of the
  // float with the low two of them replaced by a tag (1 or 2) that tells the reader which tile the value belongs to (a
  // reference maximum needs no more precision; both threads of a row use the same truncated words).  The exchange of the
  // maxima of an item's first tile borrows the slot that is idle at that moment and leaves it cleared.
  uint16_t xmax[2][2][128];
  float row_l[2][128];                           // [half][row]: row sum of a finished item, for the other half's epilogue
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

// 32-byte store (a whole sector per lane).  `p` must be 32-byte aligned.
__device__ __forceinline__ void st_global_32B(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e, uint32_t f,
                                              uint32_t g, uint32_t h) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e),
               "r"(f), "r"(g), "r"(h) : "memory");
}
// Mailbox words: the upper half of a float (tag in its low two bits), read back as a float with a zero lower half.
__device__ __forceinline__ uint32_t ld_mailbox(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.volatile.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
  return static_cast<uint32_t>(v) << 16;
}
__device__ __forceinline__ void st_mailbox(uint32_t addr, uint32_t word) {
  asm volatile("st.volatile.shared.u16 [%0], %1;" ::"r"(addr), "h"(static_cast<uint16_t>(word >> 16)) : "memory");
}

// Barrier among the threads that share an mbarrier initialised with their number; `n` counts this thread's uses.  Unlike
// bar.sync the wait is bounded, so warps that have given up (abort) cannot leave the others hanging.
__device__ __forceinline__ bool group_sync(uint64_t* bar, uint32_t& n, volatile int* abort_flag) {
  mbar_arrive(bar);
  const bool ok = mbar_wait(bar, n & 1u, abort_flag);
  ++n;
  return ok;
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

// Epilogue of a finished item, by the eight softmax warps (all 256 threads, out of line: it runs once per item and
// must not cost the tile loop registers): the two halves of a row add their row sums, each reads 64 columns of the
// accumulator and writes them out (final bf16 rows of a verification item, fp32 partials of a stacked item).  An item
// marked in C.overflow is recomputed exactly on the CUDA cores instead.  `acc` is the item's accumulator / row-sum
// set and `acc_parity` the parity of its o_full phase; an item without tiles (no visible key) has neither.
__device__ __noinline__ void item_epilogue(const Params& P, Ctrl& C, uint32_t tmem, int slot, int acc, uint32_t acc_parity,
                                           float l_own, float m, uint32_t& n_epi, uint32_t& n_pair,
                                           volatile int* abort_flag) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int hf = warp >> 2, row = tid & 127;
  // The two halves of a row exchange their sums (one buffer: the second pair barrier keeps a thread from posting the
  // next item's sum before its partner has read this one); after the barrier of all eight warps every softmax thread
  // is past the item's tiles, so its overflow mark is final.
  C.row_l[hf][row] = l_own;
  bool ok = group_sync(&C.epi_bar, n_epi, abort_flag);
  const float l_all = l_own + C.row_l[hf ^ 1][row];
  ok = group_sync(&C.pair_bar[warp & 3], n_pair, abort_flag) && ok;
  const ItemView it = view(C.item[slot]);
  const int G = P.G;
  const int i = row / G, hl = row - i * G;
  const bool row_valid = i < it.n_tok;
  const int h = it.g * G + hl;
  const bool has_tiles = it.n_tiles > 0;
  if (has_tiles) {
    ok = mbar_wait(&C.o_full[acc], acc_parity, abort_flag) && ok;
    tc_fence_after();
  }
  ok = __all_sync(0xffffffffu, ok);
  if (ok && has_tiles && C.overflow[slot]) {
    // scores that rose by more than 2^40 from one tile to the next: the tensor-core pass holds garbage for the item
    tile_item_rows_exact(P, C.item[slot], warp, kSoftmaxWarps, lane);
  } else if (ok) {
    int64_t q_row = 0;
    int dec = 0;
    if (row_valid) {
      if (it.kind == kItemChain) q_row = it.tok0 + i;
      else { dec = it.tok0 + i; q_row = P.dec_tok[dec]; }
    }
    const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
    const float lse = l_all > 0.f ? m * P.scale + __logf(l_all) : -INFINITY;
    const bool final_out = it.slot_off < 0;
    const int64_t slot_row = final_out ? 0 : static_cast<int64_t>(row_valid ? P.dec_slot_base[dec] : 0) + it.slot_off;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
#pragma unroll
    for (int c0 = hf * 64; c0 < hf * 64 + 64; c0 += 32) {
      uint32_t orow[32];
      __syncwarp();                                         // the TMEM load below is warp-collective
      if (has_tiles) {
        tmem_ld32(tmem + lane_base + kColO + acc * kTile + c0, orow);
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
        float* dst = P.part_o + (slot_row * P.Hq + h) * kHeadDim + c0;
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
      if (final_out) { if (P.lse) P.lse[q_row * P.Hq + h] = lse; }
      else P.part_lse[slot_row * P.Hq + h] = lse;
    }
  }
  // the accumulator may be overwritten (its reads are complete) and the descriptor slot recycled
  tc_fence_before();
  __syncwarp();
  if (lane == 0) {
    if (has_tiles) mbar_arrive(&C.o_free[acc]);
    mbar_arrive(&C.item_free[slot]);
  }
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
tile_items_umma_flow_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                           const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ Params P) {
  ss::grid_dependency_enter();
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ Ctrl C;
  SS_STAMP_BEGIN(P.hdr, 2);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &C.abort_flag;

  if (tid == 0) {
    C.abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;
    for (int s = 0; s < kItemRing; ++s) { mbar_init(&C.item_ready[s], 1); mbar_init(&C.item_free[s], kSoftmaxWarps + 4); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&C.q_full[s], 1); mbar_init(&C.q_empty[s], 1);
      mbar_init(&C.o_full[s], 1); mbar_init(&C.o_free[s], kSoftmaxWarps);
    }
    for (int s = 0; s < kStagesK; ++s) { mbar_init(&C.k_full[s], 1); mbar_init(&C.k_empty[s], 1); }
    for (int s = 0; s < kStagesV; ++s) { mbar_init(&C.v_full[s], 1); mbar_init(&C.v_empty[s], 1); }
    for (int s = 0; s < 4; ++s) mbar_init(&C.pair_bar[s], 64);
    mbar_init(&C.epi_bar, kSoftmaxWarps * 32);
    for (int b = 0; b < kRing; ++b) {
      mbar_init(&C.s_full[b], 1); mbar_init(&C.p_full[b], kSoftmaxWarps * 32); mbar_init(&C.pv_done[b], 1);
    }
    fence_barrier_init();
    prefetch_tensormap(&tmap_k);
    prefetch_tensormap(&tmap_v);
    prefetch_tensormap(&tmap_q);
  }
  for (int x = tid; x < 65536 / 16; x += kUmmaThreads) reinterpret_cast<uint4*>(smem + kOffQ)[x] = make_uint4(0, 0, 0, 0);
  for (int x = tid; x < 2 * 2 * 128; x += kUmmaThreads) (&C.xmax[0][0][0])[x] = 0;    // tag 0: nothing posted
  if (tid < kItemRing) C.overflow[tid] = 0;
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

  // Running counts, advanced identically by every role: items started, items that had tiles (they select the Q buffer
  // and the accumulator), tiles processed.
  uint32_t seq = 0, uses = 0, g_tile = 0;

  // Takes the next item from the global counter into descriptor slot `dst` (one thread).
  auto fetch_item = [&](int dst) {
    int e = -1;
    if (P.hdr->status == SS_OK && !C.abort_flag) e = atomicAdd(&P.hdr->tile_counter, 1);
    if (e >= 0 && e < n_items) C.item[dst] = P.tile_items[e];
    C.item_e[dst] = e;
    C.overflow[dst] = 0;
    __threadfence_block();
    mbar_arrive(&C.item_ready[dst]);
  };
  if (tid == 0) { fetch_item(0); fetch_item(1); }
  __syncthreads();

  if (warp < kSoftmaxWarps) {
    // ===================================================== softmax + epilogue ====================================
    // Two threads per query row (= TMEM lane): thread `hf` of the pair takes score columns [64 hf, 64 hf + 64) of every
    // tile, keeps its own partial row sum and writes output columns [64 hf, 64 hf + 64).  Both derive the same
    // reference maximum: from the exact half maxima of an item's first tile (exchanged through a pair barrier) and,
    // one tile behind, from the sampled maxima that each posts for the other.
    const int hf = warp >> 2;
    const int row = tid & 127;
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    uint32_t n_pair = 0, n_epi = 0;                               // uses of the pair barrier / of the epilogue barrier
    const uint32_t xm_own = smem_u32(&C.xmax[0][hf][row]), xm_oth = smem_u32(&C.xmax[0][hf ^ 1][row]);
    bool pending = false;          // the previous item's epilogue is still to do
    int p_slot = 0, p_acc = 0;     // ... its descriptor slot and accumulator,
    uint32_t p_parity = 0;
    float p_l = 0.f, p_m = 0.f;    // ... this thread's row sum and the row's reference maximum
    bool ok = true;
    for (;;) {
      const int slot = seq % kItemRing;
      if (!mbar_wait(&C.item_ready[slot], (seq / kItemRing) & 1, abort_flag)) { ok = false; break; }
      const int e = C.item_e[slot];
      if (e < 0 || e >= n_items) break;
      const ItemView it = view(C.item[slot]);
      const int n_tiles = it.n_tiles;
      if (n_tiles == 0) {          // no key at all: zeros / -inf, written at once
        if (pending) { item_epilogue(P, C, tmem, p_slot, p_acc, p_parity, p_l, p_m, n_epi, n_pair, abort_flag); pending = false; }
        item_epilogue(P, C, tmem, slot, 0, 0, 0.f, 0.f, n_epi, n_pair, abort_flag);
        ++seq;
        continue;
      }
      const int acc = uses & 1;
      const int i = row / G;
      float m = 0.f, l = 0.f;                                     // reference maximum (0 while the row has no visible key)
      uint32_t own_post = 0;                                      // what this thread posted for the previous tile
      int limit_row = (it.kind == kItemChain) ? it.limit0 + i : it.limit0;
      if (limit_row > it.kv_end) limit_row = it.kv_end;
      const int first_masked_tile = __reduce_min_sync(0xffffffffu, max(limit_row - it.kv_begin, 0) / kTile);
      const int ragged_tile = ((it.kv_end - it.kv_begin) % kTile) ? n_tiles - 1 : -1;   // only a last tile can end early
      // Everything that depends on the tile number is carried along instead of recomputed.
      int b = g_tile & 1;                                         // S buffer of the tile
      uint32_t b_phase = (g_tile >> 1) & 1;
      uint32_t par = g_tile & 1;                                  // mailbox slot of the tile's post
      uint32_t tag = ((g_tile >> 1) & 1u) + 1u;                   // tag of the tile's post
      uint32_t tag_prev = (((g_tile - 1) >> 1) & 1u) + 1u;        // tag of the previous tile's post (slot par ^ 1)
      for (int j = 0; j < n_tiles; ++j) {
        const uint32_t gj = g_tile + j;
        const uint32_t s_col = kColS + b * kTile + hf * 64;       // this thread's 64 scores; its P goes over the first 32
        if (!mbar_wait(&C.s_full[b], b_phase, abort_flag)) ok = false;
        tc_fence_after();
        uint32_t sr[64];
        tmem_ld32(tmem + lane_base + s_col, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
        tmem_wait_ld();
        tmem_ld32(tmem + lane_base + s_col + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));

        const bool masked = j >= first_masked_tile;               // warp-uniform
        bool second_in = false;
        if (masked || j == 0) {
          tmem_wait_ld();
          tmem_pin32(*reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
          second_in = true;
          if (masked) {
            const int nvis = limit_row - (it.kv_begin + j * kTile + hf * 64);   // visible ones of this thread's columns
#pragma unroll
            for (int c = 0; c < 64; ++c)
              if (c >= nvis) sr[c] = 0xff800000u;                 // -inf
          }
        }
        // ---- reference of this tile ----------------------------------------------------------------------------------
        float alpha = 1.f;
        if (j == 0) {                                             // exact maximum of the first tile, both halves
          float e4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 64; c += 2)
            e4[(c >> 1) & 3] = max3(e4[(c >> 1) & 3], __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
          const float mine = fmaxf(fmaxf(e4[0], e4[1]), fmaxf(e4[2], e4[3]));
          // (slot par ^ 1 is idle until the post of tile gj + 1; -inf survives the truncation, 0xff80)
          const uint32_t mine_t = __float_as_uint(mine) & 0xffff0000u;
          st_mailbox(xm_own + (par ^ 1u) * (2 * 128 * 2), mine_t);
          ok = group_sync(&C.pair_bar[warp & 3], n_pair, abort_flag) && ok;
          const float mxe = fmaxf(__uint_as_float(mine_t), __uint_as_float(ld_mailbox(xm_oth + (par ^ 1u) * (2 * 128 * 2))));
          m = mxe > -INFINITY ? mxe : 0.f;
          ok = group_sync(&C.pair_bar[warp & 3], n_pair, abort_flag) && ok;
          st_mailbox(xm_own + (par ^ 1u) * (2 * 128 * 2), 0u);
        } else {                                                  // lagged: the sampled maxima of the previous tile
          const uint32_t src = xm_oth + (par ^ 1u) * (2 * 128 * 2);
          uint32_t other = ld_mailbox(src);
          if (((other >> 16) & 3u) != tag_prev) {                 // the other half is still inside the previous tile
            const long long t0 = clock64();
            while ((((other = ld_mailbox(src)) >> 16) & 3u) != tag_prev) {
              if (*abort_flag || clock64() - t0 > kWaitCycles) { *abort_flag = 1; ok = false; break; }
            }
          }
          const float mx_prev = fmaxf(__uint_as_float(own_post), __uint_as_float(other));
          if (mx_prev > m + lazy_raw) {
            alpha = ex2((m - mx_prev) * cl2);
            m = mx_prev;
            l *= alpha;
          }
        }
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
        float sum4[4];
        unpack2(sum2[0], sum4[0], sum4[1]);
        unpack2(sum2[1], sum4[2], sum4[3]);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float tile_sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        // post this tile's sampled maximum for the other half (finite or -inf; the tag marks the tile)
        own_post = (__float_as_uint(mx) & 0xfffc0000u) | (tag << 16);
        st_mailbox(xm_own + par * (2 * 128 * 2), own_post);
        if (!(tile_sum <= jump_sum)) C.overflow[slot] = 1;       // beyond the lagged reference's range: exact pass needed
        l += tile_sum;
        const bool ragged = j == ragged_tile;
        // (only the first half's warps vote: they own O and the V tail, and a vote per tile in every warp costs 3 %)
        const bool rare = hf == 0 && (__any_sync(0xffffffffu, alpha != 1.f && j > 0) || ragged);
        if (rare) {
          if (__any_sync(0xffffffffu, alpha != 1.f && j > 0)) {   // rescale O (warp-collective TMEM access)
            ok = mbar_wait(&C.pv_done[(gj - 1) & 1], ((gj - 1) >> 1) & 1, abort_flag) && ok;
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
              uint32_t o0[32];
              tmem_ld32(tmem + lane_base + kColO + acc * kTile + c0, o0);
              tmem_wait_ld();
#pragma unroll
              for (int x = 0; x < 32; ++x) o0[x] = __float_as_uint(__uint_as_float(o0[x]) * alpha);
              tmem_st32(tmem + lane_base + kColO + acc * kTile + c0, o0);
            }
          }
          if (ragged) {                                           // zero the V rows past the end of the source
            const int n_keys = it.kv_end - (it.kv_begin + j * kTile);
            const int s = gj % kStagesV;
            ok = mbar_wait(&C.v_full[s], (gj / kStagesV) & 1, abort_flag) && ok;
            uint8_t* vs = smem + kOffV + s * kStageBytes;
            const int n_chunks = (kTile - n_keys) * 16;           // 16-byte chunks to clear (both halves)
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
        b ^= 1;
        if (b == 0) b_phase ^= 1u;
        tag_prev = tag;
        if (par) tag ^= 3u;                                       // (the tag changes with every second tile: 1 <-> 2)
        par ^= 1u;
        // The previous item's rows are written out here, after this item's first tile has been handed to the tensor
        // pipe: its last P V completed long ago, and the pipe has this item's next products to work on meanwhile.
        if (j == 0 && pending) {
          item_epilogue(P, C, tmem, p_slot, p_acc, p_parity, p_l, p_m, n_epi, n_pair, abort_flag);
          pending = false;
        }
      }
      // ---- the item's row state, for its (deferred) epilogue -----------------------------------------------------------
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      pending = true;
      p_l = l;
      p_m = m;
      p_slot = slot;
      p_acc = acc;
      p_parity = (uses >> 1) & 1;
      ++uses;
      g_tile += n_tiles;
      ++seq;
    }
    if (pending && ok) item_epilogue(P, C, tmem, p_slot, p_acc, p_parity, p_l, p_m, n_epi, n_pair, abort_flag);
  }
  else if (warp < kSoftmaxWarps + 2) {
    // ===================================================== TMA producers =========================================
    // Warp kSoftmaxWarps streams the K tiles, the next warp the V tiles, item after item, each as far ahead of its
    // consumer as its ring allows.  What an item needs before its first copy can be issued - its descriptor, the page
    // segments of its chain (dependent loads up the tree), the page ids of its first four tiles - takes a few
    // microseconds, more than the ring covers; so it is prepared one item ahead, in the middle of the current item's
    // stream (after its first block of tiles, when the warp would be waiting for ring space anyway), and kept in
    // registers: lane d of the warp holds segment d of the chain, two sets (this item / the next).
    const int which = warp - kSoftmaxWarps;                    // 0: K, 1: V
    const int n_stages = which ? kStagesV : kStagesK;
    const CUtensorMap* tm = which ? &tmap_v : &tmap_k;
    uint64_t* full = which ? C.v_full : C.k_full;
    uint64_t* empty = which ? C.v_empty : C.k_empty;
    uint8_t* ring = smem + (which ? kOffV : kOffK);
    int prod_stage = 0;       // ring stage of the next tile to issue, and how often the ring has wrapped
    uint32_t prod_wraps = 0;  //   (kept as counters: a modulo by a stage count that differs per warp is a division per tile)

    struct Prep {             // what the warp holds about an item before streaming it
      ItemView v;
      int valid;              // 0: the item list has ended (or the wait for the descriptor ran out)
      int n_seg;              // page segments of the source: one per non-empty chain node (stacked item: 1)
      int seg_first;          // lane d: first virtual page of segment d (lane n_seg: total pages)
      int seg_off;            // lane d: index into node_pages of segment d's first page
      int coord0;             // lane 8 t + pg: row coordinate of page pg of tile t (the first block of four tiles)
    };
    // row coordinate (in the pool viewed as rows of 128 elements) of page `pg` of tile j's (page, kv head) block
    auto page_coord = [&](const Prep& p, int j, int pg) -> int {
      const ItemView& v = p.v;
      int vp = -1;
      if (j < v.n_tiles) {
        const int pos0 = v.kv_begin + j * kTile;
        const int n_pages = (min(kTile, v.kv_end - pos0) + kPage - 1) / kPage;
        if (pg < n_pages) vp = pos0 / kPage + pg;
      }
      // segment of the page: the shuffles are executed by every lane (vp differs per lane, -1: no such page)
      int d = 0;
      for (int x = 1; x < p.n_seg; ++x) {
        const int f = __shfl_sync(0xffffffffu, p.seg_first, x);
        if (vp >= f) d = x;
      }
      const int first = __shfl_sync(0xffffffffu, p.seg_first, d);
      const int off = __shfl_sync(0xffffffffu, p.seg_off, d);
      if (vp < 0) return 0;
      const int64_t phys = P.node_pages[off + (vp - first)];
      return static_cast<int>((phys * P.page_stride + static_cast<int64_t>(v.g) * P.head_stride) >> 7);
    };
    // Prepares item `s` (whole warp; false if a wait ran out).  The chain walk is done by every lane alike (uniform
    // loads), lane d keeps segment d.
    auto prepare = [&](uint32_t s, Prep& p) -> bool {
      p.valid = 0;
      const int slot = s % kItemRing;
      if (!mbar_wait(&C.item_ready[slot], (s / kItemRing) & 1, abort_flag)) return false;
      const int e = C.item_e[slot];
      if (e < 0 || e >= n_items) return true;
      p.v = view(C.item[slot]);
      p.valid = 1;
      p.seg_first = 0x7fffffff;
      p.seg_off = 0;
      const TileItem& ti = C.item[slot];
      int n_seg = ti.n_seg;
      if (n_seg >= 0) {                         // the planner has laid the segments out in the descriptor
        if (lane < n_seg) {
          p.seg_first = lane == 0 ? 0 : ti.seg_first[lane - 1];
          p.seg_off = ti.seg_off[lane];
        }
      } else {                                  // a chain deeper than the descriptor holds: walk it
        n_seg = 0;
        int chain[SS_MAX_DEPTH];
        int d = 0;
        for (int a = p.v.node; a >= 0 && d < SS_MAX_DEPTH; a = P.node_parent[a]) chain[d++] = a;
        int first = 0;
        for (int c = d - 1; c >= 0; --c) {
          const int n = chain[c];
          const int np = (P.node_kv_len[n] + kPage - 1) / kPage;
          if (np == 0) continue;
          if (lane == n_seg) { p.seg_first = first; p.seg_off = static_cast<int>(P.node_page_offsets[n]); }
          first += np;
          ++n_seg;
        }
      }
      p.n_seg = n_seg;
      p.coord0 = page_coord(p, lane >> 3, lane & 7);
      return true;
    };
    // tiles [j_begin, j_end) of the prepared item; calls follow one another in tile order, so the stage counters run
    // on.  `cur` holds the page coordinates of the block that starts at j_begin (lane 8 t + pg).
    auto stream_tiles = [&](const Prep& p, int j_begin, int j_end, int cur) -> bool {
      const ItemView& v = p.v;
      bool ok = true;
      // The page ids of four tiles are fetched with one load per lane, a whole block ahead of their use; the lanes hand
      // them to ONE elected lane by shuffles, and that lane issues all copies of the block in straight-line code
      // (bulk-tensor copies are issued from uniform registers).
      for (int j0 = j_begin; j0 < j_end && ok; j0 += 4) {
        const int nxt = (j0 + 4 < j_end) ? page_coord(p, j0 + 4 + (lane >> 3), lane & 7) : 0;
        const int n_blk = min(4, j_end - j0);
        int y[4][8];                                           // (every lane gets all 32: the elected one uses them)
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
          for (int pg = 0; pg < 8; ++pg) y[t][pg] = __shfl_sync(0xffffffffu, cur, t * 8 + pg);
        if (elect_one()) {
          int s = prod_stage;
          uint32_t u = prod_wraps;
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            if (t >= n_blk) break;
            const int pos0 = v.kv_begin + (j0 + t) * kTile;
            const int n_pages = (min(kTile, v.kv_end - pos0) + kPage - 1) / kPage;
            if (u > 0 && !mbar_wait(&empty[s], (u - 1) & 1, abort_flag)) { ok = false; break; }
            mbar_arrive_expect_tx(&full[s], static_cast<uint32_t>(n_pages) * 4096u);
            uint8_t* dst = ring + s * kStageBytes;
#pragma unroll
            for (int pg = 0; pg < kTile / kPage; ++pg) {
              if (pg < n_pages) {
                tma_load_4d(dst + pg * 4096, tm, 0, 0, 0, y[t][pg] >> 3, &full[s]);   // the whole (page, head) block
              }
            }
            if (++s == n_stages) { s = 0; ++u; }
          }
        }
        __syncwarp();
        ok = __all_sync(0xffffffffu, ok);
        prod_stage += n_blk;                                   // every lane keeps the counters
        while (prod_stage >= n_stages) { prod_stage -= n_stages; ++prod_wraps; }
        cur = nxt;
      }
      return ok;
    };
    // Q buffer `u & 1` is recycled for the u-th item that has tiles: its previous user's Q K^T products must be done
    auto q_buffer_free = [&](uint32_t u) -> bool {
      return u < 2 || mbar_wait(&C.q_empty[u & 1], ((u >> 1) - 1) & 1, abort_flag);
    };
    // Stacked items: asynchronous copy of the (gathered) Q rows into Q buffer `buf` (UMMA K-major layout with the
    // 128-byte swizzle; rows past the item's last one are zero-filled)
    auto q_gather_start = [&](const ItemView& v, int buf) {
      const uint32_t dst0 = smem_u32(smem + kOffQ + buf * 32768);
#pragma unroll 1
      for (int row = lane; row < 128; row += 32) {
        const int i = row / G, hl = row - i * G;
        const bool row_valid = i < v.n_tok;
        int64_t q_src = 0;
        if (row_valid) q_src = P.dec_src[v.tok0 + i];
        const char* src = reinterpret_cast<const char*>(P.q + (q_src * P.Hq + (v.g * G + hl)) * kHeadDim);
        const uint32_t n_src = row_valid ? 16u : 0u;             // 0 source bytes: the 16 destination bytes are zeroed
#pragma unroll
        for (int ch = 0; ch < 16; ++ch)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst0 + (ch >> 3) * 16384 + sw128_offset(row, ch & 7)),
                       "l"(src + ch * 16), "r"(n_src) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // Verification items: the Q rows are a box of the query tensor (one thread; rows of the box past the item's tokens
    // belong to other paths or are zero-filled: finite either way, and never written out)
    auto q_tma_start = [&](const ItemView& v, int buf) {
      uint8_t* dst = smem + kOffQ + buf * 32768;
      mbar_arrive_expect_tx(&C.q_full[buf], static_cast<uint32_t>(2 * 128 * G * P.tok_per_tile));
      tma_load_3d(dst, &tmap_q, 0, v.g * G, v.src0, &C.q_full[buf]);
      tma_load_3d(dst + 16384, &tmap_q, 64, v.g * G, v.src0, &C.q_full[buf]);
    };
    // Starts the Q copy of item `v` (the u-th with tiles) if it is this warp's kind; returns true if a gather is pending
    auto q_start = [&](const ItemView& v, uint32_t u, bool& ok) -> bool {
      if (v.n_tiles == 0) return false;
      if (which == 0 && v.kind == kItemChain) {
        ok = q_buffer_free(u) && ok;
        ok = __all_sync(0xffffffffu, ok);
        if (ok && elect_one()) q_tma_start(v, u & 1);
        __syncwarp();
      } else if (which == 1 && v.kind != kItemChain) {
        ok = q_buffer_free(u) && ok;
        ok = __all_sync(0xffffffffu, ok);
        if (ok) { q_gather_start(v, u & 1); return true; }
      }
      return false;
    };
    auto q_gather_finish = [&](uint32_t u) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&C.q_full[u & 1]);
    };

    bool ok = true;
    bool gather_pending = false;   // (V producer) the Q rows of the coming item are being gathered
    Prep cur, nxt;
    ok = prepare(0, cur);
    if (ok && cur.valid && q_start(cur.v, 0, ok)) q_gather_finish(0);       // Q of the very first item
    while (ok && cur.valid) {
      const ItemView& it = cur.v;
      if (lane == 0) mbar_arrive(&C.item_free[seq % kItemRing]);  // (this role holds the descriptor in registers now)
      const uint32_t u_next = uses + (it.n_tiles > 0 ? 1u : 0u);
      if (gather_pending) { q_gather_finish(uses); gather_pending = false; }   // this item's Q rows, gathered meanwhile
      // ---- the first block of this item's tiles ------------------------------------------------------------------------
      ok = stream_tiles(cur, 0, min(4, it.n_tiles), cur.coord0);
      if (!ok) break;
      // ---- descriptor of item seq + 2 (K producer): its slot was item seq + 2 - kItemRing's ------------------------------
      if (which == 0) {
        const uint32_t n = seq + 2;
        if (n >= static_cast<uint32_t>(kItemRing))
          ok = mbar_wait(&C.item_free[n % kItemRing], ((n / kItemRing) - 1) & 1, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 31) fetch_item(n % kItemRing);
      }
      // ---- the next item, prepared while this one's first tiles are consumed ---------------------------------------------
      ok = prepare(seq + 1, nxt);
      if (!ok) break;
      // ---- the rest of this item's tiles ----------------------------------------------------------------------------------
      if (it.n_tiles > 4) {
        ok = stream_tiles(cur, 4, it.n_tiles, page_coord(cur, 4 + (lane >> 3), lane & 7));
        if (!ok) break;
      }
      // ---- Q of the next item: now, not earlier - its buffer is the previous item's, whose last Q K^T completes up to
      //      three tiles after this warp has moved on to this item, and waiting for that before streaming this item's
      //      tiles would drain the ring at every item boundary --------------------------------------------------------
      if (nxt.valid) {
        gather_pending = q_start(nxt.v, u_next, ok);
        if (!ok) break;
      }
      uses = u_next;
      g_tile += it.n_tiles;
      ++seq;
      cur = nxt;
    }
  } else if (warp == kSoftmaxWarps + 2) {
    // ===================================================== S = Q K^T issuer ======================================
    if (elect_one()) {                                           // (elected, not `lane == 0`: see the producers)
      constexpr uint32_t idesc_qk = instr_desc_bf16(128, kTile, false);
      const uint64_t k_desc0 = smem_desc_sw128(smem_u32(smem + kOffK), 0, 2048);   // 8-key groups 2048 B apart
      bool ok = true;
      while (ok) {
        const int slot = seq % kItemRing;
        if (!mbar_wait(&C.item_ready[slot], (seq / kItemRing) & 1, abort_flag)) break;
        const int e = C.item_e[slot];
        if (e < 0 || e >= n_items) break;
        const ItemView it = view(C.item[slot]);
        mbar_arrive(&C.item_free[slot]);
        const int n_tiles = it.n_tiles;
        if (n_tiles > 0) {
          const int qb = uses & 1;
          const uint64_t q_desc0 = smem_desc_sw128(smem_u32(smem + kOffQ + qb * 32768), 0, 1024);
          ok = mbar_wait(&C.q_full[qb], (uses >> 1) & 1, abort_flag);
          for (int j = 0; j < n_tiles && ok; ++j) {
            const uint32_t gj = g_tile + j;
            const int s = gj % kStagesK, b = gj & 1;
            // buffer b held S / P of tile gj - 2: free once the P V product that read it has completed
            if (gj >= 2) ok = mbar_wait(&C.pv_done[b], ((gj >> 1) - 1) & 1, abort_flag);
            ok = ok && mbar_wait(&C.k_full[s], (gj / kStagesK) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint64_t k_desc = smem_desc_advance(k_desc0, static_cast<uint32_t>(s) * kStageBytes);
            const uint32_t d_tmem = tmem + kColS + b * kTile;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              mma_bf16_ss(d_tmem, smem_desc_advance(q_desc0, (kk >> 2) * 16384 + (kk & 3) * 32),
                          smem_desc_advance(k_desc, (kk >> 2) * 1024 + (kk & 3) * 32), idesc_qk, kk > 0 ? 1u : 0u);
            mma_commit(&C.k_empty[s]);
            mma_commit(&C.s_full[b]);
          }
          if (ok) mma_commit(&C.q_empty[qb]);                    // the Q buffer may be refilled when these products are done
          ++uses;
          g_tile += n_tiles;
        }
        ++seq;
      }
    }
  } else {
    // ===================================================== O += P V issuer =======================================
    if (elect_one()) {
      constexpr uint32_t idesc_pv = instr_desc_bf16(128, kHeadDim, true);
      const uint64_t v_desc0 = smem_desc_sw128(smem_u32(smem + kOffV), 1024, 2048);   // dims 64..127 1024 B on, 8-key groups 2048 B apart
      bool ok = true;
      while (ok) {
        const int slot = seq % kItemRing;
        if (!mbar_wait(&C.item_ready[slot], (seq / kItemRing) & 1, abort_flag)) break;
        const int e = C.item_e[slot];
        if (e < 0 || e >= n_items) break;
        const ItemView it = view(C.item[slot]);
        mbar_arrive(&C.item_free[slot]);
        const int n_tiles = it.n_tiles;
        if (n_tiles > 0) {
          const int acc = uses & 1;
          // accumulator `acc` was item (uses - 2)'s: free once its epilogue has read it
          if (uses >= 2) ok = mbar_wait(&C.o_free[acc], ((uses >> 1) - 1) & 1, abort_flag);
          const uint32_t o_tmem = tmem + kColO + acc * kTile;
          for (int j = 0; j < n_tiles && ok; ++j) {
            const uint32_t gj = g_tile + j;
            const int s = gj % kStagesV, b = gj & 1;
            ok = mbar_wait(&C.v_full[s], (gj / kStagesV) & 1, abort_flag) &&
                 mbar_wait(&C.p_full[b], (gj >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint64_t v_desc = smem_desc_advance(v_desc0, static_cast<uint32_t>(s) * kStageBytes);
            const uint32_t p_tmem = tmem + kColS + b * kTile;
#pragma unroll
            for (int kk = 0; kk < kTile / 16; ++kk)       // P of keys 0..63 at columns 0..31, of keys 64..127 at 64..95
              mma_bf16_ts(o_tmem, p_tmem + (kk >> 2) * 64 + (kk & 3) * 8, smem_desc_advance(v_desc, kk * 4096), idesc_pv,
                          (j > 0 || kk > 0) ? 1u : 0u);
            mma_commit(&C.v_empty[s]);
            mma_commit(&C.pv_done[b]);
            if (j + 1 == n_tiles) mma_commit(&C.o_full[acc]);
          }
          ++uses;
          g_tile += n_tiles;
        }
        ++seq;
      }
    }
  }

  // ---- teardown --------------------------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (C.abort_flag) {
    if (tid == 0) set_status(&P.hdr->status, SS_ERR_TIMEOUT);
    const long long t0 = clock64();                 // let copies / MMAs that are still in flight land
    while (clock64() - t0 < 4000000LL) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == kSoftmaxWarps) tmem_dealloc(tmem, kTmemCols);
  SS_STAMP_END(P.hdr, 3);
}

}  // namespace flow

int32_t launch_tile_items_umma(const Params& P, cudaStream_t st, int sm_count);   // the 64-key kernel (attn_umma.cu)

int32_t launch_tile_items_umma_flow(const Params& P, cudaStream_t st, int sm_count) {
  using namespace flow;
  // One bulk-tensor copy per (page, kv head) block needs the blocks to start on 8-row boundaries of the pool (rows of
  // 256 bytes); any other pool layout goes to the kernel that copies the two 64-dim halves of a block separately.
  if (P.page_stride % 1024 || P.head_stride % 1024) return launch_tile_items_umma(P, st, sm_count);
  static bool configured[kDeviceSlots] = {false};     // the attribute belongs to the (function, device) pair
  const int dev_slot = current_device_slot();
  if (dev_slot < 0 || !configured[dev_slot]) {
    if (cudaFuncSetAttribute(tile_items_umma_flow_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem) !=
        cudaSuccess) {
      (void)cudaGetLastError();
      return SS_ERR_CUDA;
    }
    if (dev_slot >= 0) configured[dev_slot] = true;
  }
  const int64_t rows = ((P.num_pages > 0 ? P.num_pages - 1 : 0) * P.page_stride + (P.Hkv - 1) * P.head_stride) / 128 + kPage;
  if (rows >= 0x7fffffffLL) return SS_ERR_UNSUPPORTED;
  CUtensorMap tk, tv, tq;
  if (!tmap::encode_kv_block_bf16(&tk, P.k_pool, static_cast<uint64_t>(rows)) ||
      !tmap::encode_kv_block_bf16(&tv, P.v_pool, static_cast<uint64_t>(rows)))
    return SS_ERR_CUDA;
  const int64_t q_rows = P.q_src_offsets ? P.q_src_rows : P.total_q;
  if (!tmap::encode_q_bf16(&tq, P.q, static_cast<uint64_t>(P.Hq), static_cast<uint64_t>(q_rows > 0 ? q_rows : 1),
                           static_cast<uint32_t>(P.G), static_cast<uint32_t>(P.tok_per_tile)))
    return SS_ERR_CUDA;
  SS_LAUNCH(tile_items_umma_flow_kernel, sm_count, kUmmaThreads, kUmmaSmem, st, tk, tv, tq, P);
  return SS_OK;
}

}  // namespace attn
}  // namespace ss
