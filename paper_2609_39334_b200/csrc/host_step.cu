// ss_candidate_step_host: one pass of the whole candidate-path hot path for a caller whose per-step data lives in
// HOST memory.  It only strings together what the library already exports - asynchronous copies of the step's
// inputs into a caller-owned device arena, ss_dedup_paths, ss_gather_unique_paths, ss_tree_attention,
// ss_topk_prune, asynchronous copies of every result back - all on the caller's stream, without a host
// synchronisation, so that a caller that alternates between a few arenas and streams overlaps one step's copies
// with another step's kernels.
#include "common.cuh"

namespace ss {
namespace host_step {

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
  SS_COPY(a.q, s.q, q_bytes, H2D);
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
  const ss_attn_desc_t d = step_desc(s, a);
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
  SS_COPY(s.out, a.out, q_bytes, D2H);
  if (s.lse) SS_COPY(s.lse, a.lse, lse_bytes, D2H);
  SS_COPY(s.survivors, a.survivors, P * static_cast<size_t>(s.top_k) * 4, D2H);
  SS_COPY(s.keep, a.keep, N, D2H);
  SS_COPY(s.device_status, a.attn_ws, sizeof(int32_t), D2H);     // first word of the attention workspace
  return SS_OK;
}
