// Host-side tensor-map encoding and ss_debug_umma_tile: one 128 x N x K bf16 tile product on the tcgen05 tensor
// cores, built from exactly the pieces the attention tile kernel uses (thread-written swizzled A operand, TMA-loaded
// swizzled B operand in 16-row boxes, K-major and MN-major shared-memory descriptors, TMEM accumulator read-out).
#include "umma.cuh"

namespace ss {
namespace tmap {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      (void)cudaGetLastError();
  }
  return fn;
}

bool encode_2d_bf16(CUtensorMap* out, const void* base, uint64_t row_elems, uint64_t rows, uint64_t pitch_bytes,
                    uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {row_elems, rows};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// K / V pool viewed as rows of 128 bf16 (256 bytes).  One box = 16 consecutive rows (one page of one kv head) x all
// 128 dims, delivered as the tensor-core operand layout wants it: for each group of 8 rows, first the 8 x 128-byte
// rows of dims 0..63 (one 1024-byte swizzle atom), then those of dims 64..127.  Dimensions, innermost first:
// 64 dims (2 B apart), 8 rows (256 B), 2 halves of the row (128 B), groups of 8 rows (2048 B); the coordinate of a box
// is (0, 0, 0, first row / 8).  The strides are not monotonic (the third is smaller than the second): the rows of a
// half are gathered before the halves are.
bool encode_kv_block_bf16(CUtensorMap* out, const void* base, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {64, 8, 2, rows / 8};
  const cuuint64_t strides[3] = {256, 128, 2048};
  const cuuint32_t box[4] = {64, 8, 2, 2};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Query rows: q viewed as [token][q head][128] bf16; boxes of 64 dims x `heads` heads x `tokens` tokens land in shared
// memory as consecutive 128-byte rows (token-major, then head) with the 128-byte swizzle.
bool encode_q_bf16(CUtensorMap* out, const void* base, uint64_t q_heads, uint64_t tokens_total, uint32_t heads,
                   uint32_t tokens) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, q_heads, tokens_total};
  const cuuint64_t strides[2] = {256, q_heads * 256};
  const cuuint32_t box[3] = {64, heads, tokens};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tmap

namespace umma {

__global__ void __launch_bounds__(128) umma_tile_test_kernel(const __grid_constant__ CUtensorMap tmap_b,
                                                             const __nv_bfloat16* __restrict__ a, float* __restrict__ c,
                                                             int n, int k, int b_mn, int32_t* status) {
  ss::grid_dependency_enter();
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ uint64_t bar_tma, bar_mma;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5;
  uint8_t* sA = smem;                                   // [k/64][128 rows][128 B]
  uint8_t* sB = smem + (k / 64) * 16384;                // K-major: [k/64][n rows][128 B]; MN-major: [n/64][k rows][128 B]
  if (tid == 0) {
    abort_flag = (smem_u32(smem) & 1023u) ? 1 : 0;      // the swizzle needs 1024-byte aligned tiles
    mbar_init(&bar_tma, 1);
    mbar_init(&bar_mma, 1);
    fence_barrier_init();
  }
  if (warp == 0) tmem_alloc(&tmem_slot, 128);
  // A: thread r copies row r, 16-byte chunks to their swizzled places
  for (int ch = 0; ch < k / 8; ++ch) {
    const uint4 v = *reinterpret_cast<const uint4*>(a + static_cast<size_t>(tid) * k + ch * 8);
    *reinterpret_cast<uint4*>(sA + (ch >> 3) * 16384 + sw128_offset(tid, ch & 7)) = v;
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  bool ok = abort_flag == 0;
  if (tid == 0 && ok) {
    mbar_arrive_expect_tx(&bar_tma, static_cast<uint32_t>(n) * k * 2);
    if (!b_mn) {
      for (int kc = 0; kc < k / 64; ++kc)
        for (int r0 = 0; r0 < n; r0 += 16) tma_load_2d(sB + kc * (n * 128) + r0 * 128, &tmap_b, kc * 64, r0, &bar_tma);
    } else {
      for (int h = 0; h < n / 64; ++h)
        for (int r0 = 0; r0 < k; r0 += 16) tma_load_2d(sB + h * (k * 128) + r0 * 128, &tmap_b, h * 64, r0, &bar_tma);
    }
    ok = mbar_wait(&bar_tma, 0, &abort_flag);
    if (ok) {
      tc_fence_after();
      const uint32_t idesc = instr_desc_bf16(128, n, b_mn != 0);
      const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
      for (int kk = 0; kk < k / 16; ++kk) {
        const uint64_t ad = smem_desc_sw128(a0 + (kk >> 2) * 16384 + (kk & 3) * 32, 0, 1024);
        const uint64_t bd = b_mn ? smem_desc_sw128(b0 + kk * 2048, static_cast<uint32_t>(k) * 128, 1024)
                                 : smem_desc_sw128(b0 + (kk >> 2) * (n * 128) + (kk & 3) * 32, 0, 1024);
        mma_bf16_ss(tmem, ad, bd, idesc, kk > 0 ? 1u : 0u);
      }
    }
    mma_commit(&bar_mma);                               // also arrives when nothing was issued
  }
  __syncthreads();
  ok = abort_flag == 0 && mbar_wait(&bar_mma, 0, &abort_flag);
  tc_fence_after();
  if (ok) {
    for (int c0 = 0; c0 < n; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(tmem + (static_cast<uint32_t>(warp * 32) << 16) + c0, r);
      tmem_wait_ld();
#pragma unroll
      for (int j = 0; j < 32; ++j) c[static_cast<size_t>(tid) * n + c0 + j] = __uint_as_float(r[j]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 128);
  if (tid == 0) *status = abort_flag ? SS_ERR_TIMEOUT : SS_OK;
}

// The bounded wait on a barrier that nothing completes: must return false after its limit, with the abort flag set.
__global__ void __launch_bounds__(64) bounded_wait_test_kernel(int32_t* status) {
  ss::grid_dependency_enter();
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  // thread 0 runs into the limit itself; thread 32 is released by the flag thread 0 raises (or by its own limit)
  bool gave_up = true;
  if (threadIdx.x == 0 || threadIdx.x == 32) gave_up = !mbar_wait(&bar, 0, &abort_flag);
  const long long dt = clock64() - t0;
  const int all_gave_up = __syncthreads_and(gave_up ? 1 : 0);
  if (threadIdx.x == 0) {
    status[0] = (all_gave_up && abort_flag != 0) ? SS_ERR_TIMEOUT : SS_OK;
    status[1] = static_cast<int32_t>(dt / 1000000);
  }
}

}  // namespace umma
}  // namespace ss

extern "C" int32_t ss_debug_bounded_wait(int32_t* status_out, void* stream) {
  using namespace ss;
  if (!status_out) return SS_ERR_INVALID_ARG;
  SS_LAUNCH(umma::bounded_wait_test_kernel, 1, 64, 0, as_stream(stream), status_out);
  return SS_OK;
}

extern "C" int32_t ss_debug_umma_tile(const void* a_bf16, const void* b_bf16, float* c, int32_t n, int32_t k,
                                      int32_t b_is_mn_major, int32_t* status_out, void* stream) {
  using namespace ss;
  if (!a_bf16 || !b_bf16 || !c || !status_out) return SS_ERR_INVALID_ARG;
  if ((n != 64 && n != 128) || k < 64 || k > 256 || k % 64) return SS_ERR_UNSUPPORTED;
  CUtensorMap tm;
  const bool enc = b_is_mn_major ? tmap::encode_2d_bf16(&tm, b_bf16, n, k, static_cast<uint64_t>(n) * 2, 16)
                                 : tmap::encode_2d_bf16(&tm, b_bf16, k, n, static_cast<uint64_t>(k) * 2, 16);
  if (!enc) return SS_ERR_CUDA;
  const size_t smem = static_cast<size_t>(k / 64) * 16384 + static_cast<size_t>(n) * k * 2;
  if (cudaFuncSetAttribute(umma::umma_tile_test_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(smem)) != cudaSuccess) {
    (void)cudaGetLastError();
    return SS_ERR_CUDA;
  }
  SS_LAUNCH(umma::umma_tile_test_kernel, 1, 128, smem, as_stream(stream), tm,
            static_cast<const __nv_bfloat16*>(a_bf16), c, n, k, b_is_mn_major, status_out);
  return SS_OK;
}
