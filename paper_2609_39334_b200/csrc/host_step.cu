// ss_candidate_step_host: one pass of the whole candidate-path hot path for a caller whose per-step data lives in
// HOST memory.  It only strings together what the library already exports - asynchronous copies of the step's
// inputs into a caller-owned device arena, ss_dedup_paths, ss_gather_unique_paths, ss_tree_attention,
// ss_topk_prune, asynchronous copies of every result back - all on the caller's stream, without a host
// synchronisation, so that a caller that alternates between a few arenas and streams overlaps one step's copies
// with another step's kernels.
//
// Rows nobody reads do not cross the bus: a duplicate candidate gets no forward pass (paper, Section "Computation
// Deduplication"), so it has no query and no output of its own.  When the caller's q / out / lse buffers are
// page-locked AND mapped (cudaHostAlloc / cudaHostRegister memory: the device can address them), the token ids go
// first, the paths are deduplicated, and only then two small copy kernels move the query rows of the UNIQUE paths in
// (read straight from the host buffer) and, after the attention, the live rows of out / lse back (written straight
// into the host buffer) - how many rows those are is only known on the device, which is why kernels do it and not
// cudaMemcpyAsync.  The copy kernels are a few persistent blocks, and the attention call is told to leave as many
// SMs free (ss_attn_desc_t::max_sms): its tile and leaf blocks need an SM to themselves, and would otherwise wait
// for a copy block that runs for as long as the bus takes.  Buffers that are not mapped take the plain path: every
// logical candidate's rows are copied with cudaMemcpyAsync.
#include "common.cuh"

namespace ss {
namespace host_step {

constexpr int kCopyBlocks = 8;       // persistent blocks per copy kernel
constexpr int kCopyThreads = 512;
constexpr int kGatherBatch = 128;    // paths whose descriptors a block stages at a time

// Query rows of the live unique paths, host -> device: path u's rows [u_q_src[u], + T) of the caller's buffer become
// rows [u_q_offsets[u], + T) of the compact device buffer (a path's rows are contiguous on both sides; a batch of
// consecutive paths is contiguous on the device side).  16-byte chunks, several in flight per thread.
__global__ void __launch_bounds__(kCopyThreads)
gather_q_from_host_kernel(const uint4* __restrict__ q_host, uint4* __restrict__ q_dev, const int32_t* __restrict__ num_unique,
                          int32_t n_paths, const int64_t* __restrict__ u_q_offsets, const int64_t* __restrict__ u_q_src,
                          int64_t row_chunks, int32_t* __restrict__ batch_counter) {
  ss::grid_dependency_enter();
  __shared__ int64_t s_off[kGatherBatch + 1], s_src[kGatherBatch];
  __shared__ int s_batch;
  int live = *num_unique;
  live = live < 0 ? 0 : (live > n_paths ? n_paths : live);
  for (;;) {
    __syncthreads();
    if (threadIdx.x == 0) s_batch = atomicAdd(batch_counter, 1);
    __syncthreads();
    const int p0 = s_batch * kGatherBatch;
    if (p0 >= live) break;
    const int np = min(kGatherBatch, live - p0);
    for (int i = threadIdx.x; i <= np; i += blockDim.x) {
      s_off[i] = u_q_offsets[p0 + i];
      if (i < np) s_src[i] = u_q_src[p0 + i];
    }
    __syncthreads();
    const int64_t row0 = s_off[0];
    const int64_t n_chunks = (s_off[np] - row0) * row_chunks;
    uint4* dst = q_dev + row0 * row_chunks;
    for (int64_t c0 = threadIdx.x; c0 < n_chunks; c0 += 4LL * blockDim.x) {
      uint4 v[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int64_t c = c0 + static_cast<int64_t>(x) * blockDim.x;
        if (c >= n_chunks) break;
        const int64_t row = row0 + c / row_chunks;
        int lo = 0, hi = np;                               // path of the batch that owns the row
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (s_off[mid] <= row) lo = mid; else hi = mid;
        }
        v[x] = q_host[(s_src[lo] + (row - s_off[lo])) * row_chunks + c % row_chunks];
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int64_t c = c0 + static_cast<int64_t>(x) * blockDim.x;
        if (c < n_chunks) dst[c] = v[x];
      }
    }
  }
}

// The live rows of out / lse, device -> host: rows [0, u_q_offsets[U]) of the compact device buffers.
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
  for (int64_t c0 = tid; c0 < n_out; c0 += 4 * nt) {
    uint4 v[4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
      if (c0 + x * nt < n_out) v[x] = out_dev[c0 + x * nt];
#pragma unroll
    for (int x = 0; x < 4; ++x)
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
  int32_t* copy_counter;             // batch counter of the query gather (zeroed every step)
  // workspaces of the three calls
  void* dedup_ws; size_t dedup_ws_bytes;
  void* attn_ws; size_t attn_ws_bytes;
  void* topk_ws; size_t topk_ws_bytes;
  size_t total;
};

static size_t at_least_one(int64_t n) { return static_cast<size_t>(n > 0 ? n : 1); }

// The attention descriptor of this step: the caller's resident fields + the staged per-path arrays.
// `compact_q`: the device buffer holds the unique paths' rows at u_q_offsets (gathered from the host); otherwise it
// holds every logical candidate's rows and the attention reads them in place through u_q_src.
static ss_attn_desc_t step_desc(const ss_host_step_t& s, const Arena& a, bool compact_q = false, int max_sms = 0) {
  ss_attn_desc_t d = *s.attn;
  d.num_paths = s.n_paths;
  d.num_paths_dev = a.num_unique;
  d.path_leaf_node = a.u_leaf;
  d.path_q_len = a.u_q_len;
  d.q_offsets = a.u_q_offsets;
  d.total_q = s.total_q;
  d.q_src_offsets = compact_q ? nullptr : a.u_q_src;
  d.q_src_rows = compact_q ? 0 : s.total_q;
  d.max_sms = max_sms;
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
  a->copy_counter = c.take<int32_t>(4);
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
  const size_t lse_bytes = static_cast<size_t>(s.total_q) * static_cast<size_t>(s.attn->num_q_heads) * sizeof(float);

  // ---- host -> device: the step's candidates, queries and scores ------------------------------------------------
  const cudaMemcpyKind H2D = cudaMemcpyHostToDevice, D2H = cudaMemcpyDeviceToHost;
  SS_COPY(a.tok_ids, s.tok_ids, static_cast<size_t>(s.total_tok) * 4, H2D);
  SS_COPY(a.tok_offsets, s.tok_offsets, (N + 1) * 8, H2D);
  if (s.ctx_key) SS_COPY(a.ctx_key, s.ctx_key, N * 8, H2D);
  if (s.slot_in) SS_COPY(a.slot_in, s.slot_in, N * 4, H2D);
  SS_COPY(a.path_leaf_node, s.path_leaf_node, N * 4, H2D);
  SS_COPY(a.path_q_len, s.path_q_len, N * 4, H2D);
  SS_COPY(a.q_offsets, s.q_offsets, (N + 1) * 8, H2D);
  // mapped q / out / lse: only the unique paths' rows cross the bus (see the top of the file)
  void *q_map = nullptr, *out_map = nullptr, *lse_map = nullptr;
  bool slim = s.total_q > 0 && s.n_paths > 0 && row * sizeof(__nv_bfloat16) % 16 == 0;
  if (slim && (cudaHostGetDevicePointer(&q_map, const_cast<void*>(s.q), 0) != cudaSuccess ||
               cudaHostGetDevicePointer(&out_map, s.out, 0) != cudaSuccess ||
               (s.lse && cudaHostGetDevicePointer(&lse_map, s.lse, 0) != cudaSuccess))) {
    (void)cudaGetLastError();
    slim = false;
  }
  int dev_sms = 0;
  if (slim) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&dev_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        dev_sms <= 4 * kCopyBlocks) {
      (void)cudaGetLastError();
      slim = false;
    }
  }
  if (slim) {
    if (cudaMemsetAsync(a.copy_counter, 0, 16, st) != cudaSuccess) { (void)cudaGetLastError(); return SS_ERR_CUDA; }
  } else {
    SS_COPY(a.q, s.q, q_bytes, H2D);
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
  const int64_t row_chunks = static_cast<int64_t>(row * sizeof(__nv_bfloat16) / 16);
  if (slim)
    SS_LAUNCH(gather_q_from_host_kernel, kCopyBlocks, kCopyThreads, 0, st, static_cast<const uint4*>(q_map),
              static_cast<uint4*>(a.q), static_cast<const int32_t*>(a.num_unique), s.n_paths,
              static_cast<const int64_t*>(a.u_q_offsets), static_cast<const int64_t*>(a.u_q_src), row_chunks, a.copy_counter);
  // (two copy kernels of other steps may be running beside this step's attention: their SMs are left alone)
  const ss_attn_desc_t d = step_desc(s, a, slim, slim ? dev_sms - 2 * kCopyBlocks : 0);
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
  if (slim) {
    SS_LAUNCH(rows_to_host_kernel, kCopyBlocks, kCopyThreads, 0, st, static_cast<const uint4*>(a.out),
              static_cast<uint4*>(out_map), reinterpret_cast<const uint4*>(a.lse), static_cast<uint4*>(lse_map),
              static_cast<const int32_t*>(a.num_unique), s.n_paths, static_cast<const int64_t*>(a.u_q_offsets), row_chunks,
              static_cast<int64_t>(s.attn->num_q_heads) * 4);
  } else {
    SS_COPY(s.out, a.out, q_bytes, D2H);
    if (s.lse) SS_COPY(s.lse, a.lse, lse_bytes, D2H);
  }
  SS_COPY(s.survivors, a.survivors, P * static_cast<size_t>(s.top_k) * 4, D2H);
  SS_COPY(s.keep, a.keep, N, D2H);
  SS_COPY(s.device_status, a.attn_ws, sizeof(int32_t), D2H);     // first word of the attention workspace
  return SS_OK;
}
