// ss_candidate_step_host: one pass of the whole candidate-path hot path for a caller whose per-step data lives in
// HOST memory.  It only strings together what the library already exports - asynchronous copies of the step's
// inputs into a caller-owned device arena, ss_dedup_paths, ss_gather_unique_paths, ss_tree_attention,
// ss_topk_prune, asynchronous copies of every result back - all on the caller's stream, without a host
// synchronisation, so that a caller that alternates between a few arenas and streams overlaps one step's copies
// with another step's kernels.
//
// Rows nobody reads need not come back over the bus: a duplicate candidate gets no forward pass (paper, Section
// "Computation Deduplication"), so it has no output of its own.  With SS_STEP_COMPACT_TRANSFERS, and out / lse
// page-locked and mapped into the device's address space, only the live rows of out / lse - the first
// u_q_offsets[num_unique], a number only the device knows - are returned, by a small kernel that writes them
// straight into the host buffers.  The query rows still go in whole, with one cudaMemcpyAsync: fetching only the
// unique paths' rows was measured and is not kept - as one copy per run of unique paths (after a host wait for the
// deduplication) the ~2700 copies of a C5 step cost more than the 20 % of the bytes they save (each costs about as
// much bus time as the 512 KB gap it skips, and the wait keeps the steps from overlapping: 135 ms per step against
// 98 ms), and as a kernel reading mapped host memory the two directions together reach only 56-80 GB/s against the
// 96 GB/s of two copy engines.
#include "common.cuh"

namespace ss {
namespace host_step {

constexpr int kCopyBlocks = 8;       // persistent blocks of the copy kernel (8 reach 52 GB/s on the measured system)
constexpr int kCopyThreads = 512;

// The live rows of out / lse, device -> (mapped) host: rows [0, u_q_offsets[U]) of the compact device buffers.
__global__ void __launch_bounds__(kCopyThreads)
rows_to_host_kernel(const uint4* __restrict__ out_dev, uint4* __restrict__ out_host, const uint4* __restrict__ lse_dev,
                    uint4* __restrict__ lse_host, const int32_t* __restrict__ num_unique, int32_t n_paths,
                    const int64_t* __restrict__ u_q_offsets, int64_t out_row_chunks, int64_t lse_row_bytes) {
  ss::grid_dependency_enter();
  int live = *num_unique;
  live = live < 0 ? 0 : (live > n_paths ? n_paths : live);
  const int64_t rows = u_q_offsets[live];
  const int64_t tid = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t nt = static_cast<int64_t>(gridDim.x) * blockDim.x;
  const int64_t n_out = rows * out_row_chunks;
  for (int64_t c0 = tid; c0 < n_out; c0 += 8 * nt) {
    uint4 v[8];
#pragma unroll
    for (int x = 0; x < 8; ++x)
      if (c0 + x * nt < n_out) v[x] = out_dev[c0 + x * nt];
#pragma unroll
    for (int x = 0; x < 8; ++x)
      if (c0 + x * nt < n_out) out_host[c0 + x * nt] = v[x];
  }
  if (lse_host) {
    const int64_t n_bytes = rows * lse_row_bytes, n_lse = n_bytes / 16;
    for (int64_t c = tid; c < n_lse; c += nt) lse_host[c] = lse_dev[c];
    const float* tail_src = reinterpret_cast<const float*>(lse_dev + n_lse);       // (< 16 bytes)
    float* tail_dst = reinterpret_cast<float*>(lse_host + n_lse);
    if (tid < (n_bytes - n_lse * 16) / 4) tail_dst[tid] = tail_src[tid];
  }
}

struct Arena {                       // device-side layout of one step
  // staged inputs
  int32_t* tok_ids; int64_t* tok_offsets; int64_t* ctx_key; int32_t* slot_in;
  int32_t* path_leaf_node; int32_t* path_q_len; int64_t* q_offsets; void* q;
  float* scores; int32_t* seg_offsets;
  // results
  int32_t* canon; int32_t* path_to_unique; int32_t* unique_paths; int32_t* multiplicity; int32_t* slot_out;
  int32_t* num_unique;
  int32_t* u_leaf; int32_t* u_q_len; int64_t* u_q_offsets; int64_t* u_q_src;
  void* out; float* lse; int32_t* survivors; uint8_t* keep;
  // workspaces of the three calls
  void* dedup_ws; size_t dedup_ws_bytes;
  void* attn_ws; size_t attn_ws_bytes;
  void* topk_ws; size_t topk_ws_bytes;
  size_t total;
};

static size_t at_least_one(int64_t n) { return static_cast<size_t>(n > 0 ? n : 1); }

// The attention descriptor of this step: the caller's resident fields + the staged per-path arrays.
static ss_attn_desc_t step_desc(const ss_host_step_t& s, const Arena& a) {
  ss_attn_desc_t d = *s.attn;
  d.num_paths = s.n_paths;
  d.num_paths_dev = a.num_unique;
  d.path_leaf_node = a.u_leaf;
  d.path_q_len = a.u_q_len;
  d.q_offsets = a.u_q_offsets;
  d.total_q = s.total_q;
  d.q_src_offsets = a.u_q_src;
  d.q_src_rows = s.total_q;
  d.q = a.q;
  d.out = a.out;
  d.lse = a.lse;
  return d;
}

static int32_t carve(const ss_host_step_t& s, void* base, Arena* a) {
  Carver c(base);
  const size_t N = at_least_one(s.n_paths), P = at_least_one(s.n_segments);
  const size_t row = static_cast<size_t>(s.attn->num_q_heads) * static_cast<size_t>(s.attn->head_dim);
  a->tok_ids = c.take<int32_t>(at_least_one(s.total_tok));
  a->tok_offsets = c.take<int64_t>(N + 1);
  a->ctx_key = c.take<int64_t>(N);
  a->slot_in = c.take<int32_t>(N);
  a->path_leaf_node = c.take<int32_t>(N);
  a->path_q_len = c.take<int32_t>(N);
  a->q_offsets = c.take<int64_t>(N + 1);
  a->q = c.take<__nv_bfloat16>(at_least_one(s.total_q) * row);
  a->scores = c.take<float>(N);
  a->seg_offsets = c.take<int32_t>(P + 1);
  a->canon = c.take<int32_t>(N);
  a->path_to_unique = c.take<int32_t>(N);
  a->unique_paths = c.take<int32_t>(N);
  a->multiplicity = c.take<int32_t>(N);
  a->slot_out = c.take<int32_t>(N);
  a->num_unique = c.take<int32_t>(1);
  a->u_leaf = c.take<int32_t>(N);
  a->u_q_len = c.take<int32_t>(N);
  a->u_q_offsets = c.take<int64_t>(N + 1);
  a->u_q_src = c.take<int64_t>(N);
  a->out = c.take<__nv_bfloat16>(at_least_one(s.total_q) * row);
  a->lse = c.take<float>(at_least_one(s.total_q) * static_cast<size_t>(s.attn->num_q_heads));
  a->survivors = c.take<int32_t>(P * static_cast<size_t>(s.top_k));
  a->keep = c.take<uint8_t>(N);
  int32_t rc = ss_dedup_workspace_bytes(s.n_paths, &a->dedup_ws_bytes);
  if (rc != SS_OK) return rc;
  a->dedup_ws = c.take<char>(a->dedup_ws_bytes);
  const ss_attn_desc_t d = step_desc(s, *a);
  rc = ss_tree_attention_workspace_bytes(&d, &a->attn_ws_bytes);
  if (rc != SS_OK) return rc;
  a->attn_ws = c.take<char>(a->attn_ws_bytes);
  rc = ss_topk_workspace_bytes(s.n_paths, &a->topk_ws_bytes);
  if (rc != SS_OK) return rc;
  a->topk_ws = c.take<char>(a->topk_ws_bytes);
  a->total = c.off;
  return SS_OK;
}

static int32_t check(const ss_host_step_t* s) {
  if (!s || s->struct_size != sizeof(ss_host_step_t) || !s->attn) return SS_ERR_INVALID_ARG;
  if (s->attn->struct_size != sizeof(ss_attn_desc_t)) return SS_ERR_INVALID_ARG;
  if (s->flags & ~SS_STEP_COMPACT_TRANSFERS) return SS_ERR_INVALID_ARG;
  if (s->n_paths < 0 || s->n_segments < 0 || s->top_k < 1 || s->total_tok < 0 || s->total_q < 0)
    return SS_ERR_INVALID_ARG;
  if (s->attn->num_q_heads < 1 || s->attn->head_dim < 1) return SS_ERR_INVALID_ARG;
  return SS_OK;
}

}  // namespace host_step
}  // namespace ss

extern "C" int32_t ss_candidate_step_host_arena_bytes(const ss_host_step_t* step, size_t* out_bytes) {
  using namespace ss::host_step;
  if (!out_bytes) return SS_ERR_INVALID_ARG;
  int32_t rc = check(step);
  if (rc != SS_OK) return rc;
  Arena a;
  rc = carve(*step, nullptr, &a);        // offsets only: nothing is dereferenced
  if (rc != SS_OK) return rc;
  *out_bytes = a.total;
  return SS_OK;
}

#define SS_COPY(dst, src, bytes, kind)                                                            \
  do {                                                                                            \
    if ((bytes) > 0 && cudaMemcpyAsync((dst), (src), (bytes), (kind), st) != cudaSuccess) {       \
      (void)cudaGetLastError();                                                                   \
      return SS_ERR_CUDA;                                                                         \
    }                                                                                             \
  } while (0)

extern "C" int32_t ss_candidate_step_host(const ss_host_step_t* step, void* device_arena, size_t arena_bytes,
                                          void* stream) {
  using namespace ss;
  using namespace ss::host_step;
  int32_t rc = check(step);
  if (rc != SS_OK) return rc;
  const ss_host_step_t& s = *step;
  if (!device_arena || reinterpret_cast<uintptr_t>(device_arena) % kAlign) return SS_ERR_INVALID_ARG;
  if (!s.tok_offsets || !s.path_leaf_node || !s.path_q_len || !s.q_offsets || !s.seg_offsets || !s.canon ||
      !s.path_to_unique || !s.unique_paths || !s.multiplicity || !s.num_unique || !s.u_q_offsets || !s.survivors ||
      !s.device_status)
    return SS_ERR_INVALID_ARG;
  if ((s.slot_in == nullptr) != (s.slot_out == nullptr)) return SS_ERR_INVALID_ARG;
  if (s.n_paths > 0 && (!s.scores || !s.keep)) return SS_ERR_INVALID_ARG;
  if (s.total_tok > 0 && !s.tok_ids) return SS_ERR_INVALID_ARG;
  if (s.total_q > 0 && (!s.q || !s.out)) return SS_ERR_INVALID_ARG;
  Arena a;
  rc = carve(s, device_arena, &a);
  if (rc != SS_OK) return rc;
  if (arena_bytes < a.total) return SS_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = as_stream(stream);
  const size_t N = static_cast<size_t>(s.n_paths), P = static_cast<size_t>(s.n_segments);
  const size_t row = static_cast<size_t>(s.attn->num_q_heads) * static_cast<size_t>(s.attn->head_dim);
  const size_t q_bytes = static_cast<size_t>(s.total_q) * row * sizeof(__nv_bfloat16);

  // ---- host -> device: the step's candidates, queries and scores ------------------------------------------------
  const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
  SS_COPY(a.tok_ids, s.tok_ids, static_cast<size_t>(s.total_tok) * 4, H2D);
  SS_COPY(a.tok_offsets, s.tok_offsets, (N + 1) * 8, H2D);
  if (s.ctx_key) SS_COPY(a.ctx_key, s.ctx_key, N * 8, H2D);
  if (s.slot_in) SS_COPY(a.slot_in, s.slot_in, N * 4, H2D);
  SS_COPY(a.path_leaf_node, s.path_leaf_node, N * 4, H2D);
  SS_COPY(a.path_q_len, s.path_q_len, N * 4, H2D);
  SS_COPY(a.q_offsets, s.q_offsets, (N + 1) * 8, H2D);
  SS_COPY(a.q, s.q, q_bytes, H2D);
  // compact return: needs out / lse mapped (the kernel writes them) and whole 16-byte chunks per row
  void *out_map = nullptr, *lse_map = nullptr;
  bool compact = (s.flags & SS_STEP_COMPACT_TRANSFERS) != 0 && s.total_q > 0 && s.n_paths > 0 &&
                 row * sizeof(__nv_bfloat16) % 16 == 0;
  if (compact && (cudaHostGetDevicePointer(&out_map, s.out, 0) != cudaSuccess ||
                  (s.lse && cudaHostGetDevicePointer(&lse_map, s.lse, 0) != cudaSuccess))) {
    (void)cudaGetLastError();
    compact = false;
  }
  SS_COPY(a.scores, s.scores, N * 4, H2D);
  SS_COPY(a.seg_offsets, s.seg_offsets, (P + 1) * 4, H2D);

  // ---- the path ---------------------------------------------------------------------------------------------------
  rc = ss_dedup_paths(a.tok_ids, a.tok_offsets, s.ctx_key ? a.ctx_key : nullptr, s.slot_in ? a.slot_in : nullptr,
                      s.n_paths, s.dedup_flags, a.canon, a.path_to_unique, a.unique_paths, a.multiplicity,
                      s.slot_in ? a.slot_out : nullptr, a.num_unique, a.dedup_ws, a.dedup_ws_bytes, stream);
  if (rc != SS_OK) return rc;
  rc = ss_gather_unique_paths(a.unique_paths, a.num_unique, s.n_paths, a.path_leaf_node, a.path_q_len, a.q_offsets,
                              a.u_leaf, a.u_q_len, a.u_q_offsets, a.u_q_src, stream);
  if (rc != SS_OK) return rc;
  ss_attn_desc_t d = step_desc(s, a);
  if (compact && d.max_sms == 0) {
    // the copy kernel of the step before this one (another stream) runs for as long as the bus takes and needs SMs
    // that this step's persistent attention blocks do not hold
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
        n_sm > 4 * kCopyBlocks)
      d.max_sms = n_sm - 2 * kCopyBlocks;
    else
      (void)cudaGetLastError();
  }
  rc = ss_tree_attention(&d, a.attn_ws, a.attn_ws_bytes, stream);
  if (rc != SS_OK) return rc;
  rc = ss_topk_prune(a.scores, a.seg_offsets, s.n_segments, s.n_paths, s.top_k, a.survivors, a.keep, a.topk_ws,
                     a.topk_ws_bytes, stream);
  if (rc != SS_OK) return rc;

  // ---- device -> host: every result ------------------------------------------------------------------------------------
  SS_COPY(s.canon, a.canon, N * 4, D2H);
  SS_COPY(s.path_to_unique, a.path_to_unique, N * 4, D2H);
  SS_COPY(s.unique_paths, a.unique_paths, N * 4, D2H);
  SS_COPY(s.multiplicity, a.multiplicity, N * 4, D2H);
  if (s.slot_out) SS_COPY(s.slot_out, a.slot_out, N * 4, D2H);
  SS_COPY(s.num_unique, a.num_unique, 4, D2H);
  SS_COPY(s.u_q_offsets, a.u_q_offsets, (N + 1) * 8, D2H);
  if (compact) {
    SS_LAUNCH(rows_to_host_kernel, kCopyBlocks, kCopyThreads, 0, st, static_cast<const uint4*>(a.out),
              static_cast<uint4*>(out_map), reinterpret_cast<const uint4*>(a.lse), static_cast<uint4*>(lse_map),
              static_cast<const int32_t*>(a.num_unique), s.n_paths, static_cast<const int64_t*>(a.u_q_offsets),
              static_cast<int64_t>(row * sizeof(__nv_bfloat16) / 16), static_cast<int64_t>(s.attn->num_q_heads) * 4);
  } else {
    SS_COPY(s.out, a.out, q_bytes, D2H);
    if (s.lse) SS_COPY(s.lse, a.lse, static_cast<size_t>(s.total_q) * static_cast<size_t>(s.attn->num_q_heads) * sizeof(float), D2H);
  }
  SS_COPY(s.survivors, a.survivors, P * static_cast<size_t>(s.top_k) * 4, D2H);
  SS_COPY(s.keep, a.keep, N, D2H);
  SS_COPY(s.device_status, a.attn_ws, sizeof(int32_t), D2H);     // first word of the attention workspace
  return SS_OK;
}
