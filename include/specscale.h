/*
 * specscale.h - C ABI of the B200 (sm_100a) hot path of speculative expand-verify-select search:
 *
 *   ss_dedup_paths      computation deduplication of identical candidate paths
 *   ss_tree_attention   attention of candidate paths over a paged bf16 KV pool described by a
 *                       prefix / branch / leaf tree (decode: 1 query token per path; verification: a causal
 *                       multi-token step per path)
 *   ss_topk_prune       selection of the surviving candidates by score
 *
 * Conventions (all entry points)
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.  The library
 *     allocates no memory and keeps no state between calls; scratch comes from a caller-provided workspace
 *     whose size is returned by a pure host query (no CUDA call inside the query).
 *   - All work is enqueued on the caller's CUDA stream, passed as void* (a cudaStream_t; NULL = the legacy
 *     default stream).  No entry point synchronises the host with the device, except
 *     ss_last_device_status, which exists to do exactly that.
 *   - Host threads: calls may come from several host threads as long as calls that share a workspace, an arena or a
 *     stream do not overlap; the once-per-device set-up some calls do on first use (kernel attributes, the static
 *     scratch address) is idempotent.  The ss_profile_* diagnostics are for a single-threaded harness.
 *   - Every function returns an int32_t status.  Argument errors are detected on the host before any launch.
 *     Errors that only the device can see (an unsupported tree shape, a workspace that turns out too small
 *     for the tree, a bounded wait that expired) are recorded in the first bytes of the workspace and read
 *     back with ss_last_device_status; a call that recorded such an error leaves its outputs unspecified
 *     but never reads or writes outside the buffers it was given (as far as the index arrays are valid;
 *     SS_FLAG_VALIDATE makes the library check them too).
 *   - No exceptions, no abort, no device printf.
 */
#ifndef SPECSCALE_H_
#define SPECSCALE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------------------------------------ */
#define SS_OK 0
#define SS_ERR_INVALID_ARG 1        /* null pointer, negative size, inconsistent scalar arguments            */
#define SS_ERR_UNSUPPORTED 2        /* head_dim != 128, page_size != 16, Hq % Hkv != 0, Hq/Hkv > 128,
                                       pool rows not contiguous, tree deeper than SS_MAX_DEPTH, a shared
                                       (non-leaf) node whose length is not a multiple of the page size      */
#define SS_ERR_WORKSPACE_TOO_SMALL 3
#define SS_ERR_CUDA 4               /* a CUDA runtime / driver call failed (launch, tensor-map encode)       */
#define SS_ERR_BAD_INPUT 5          /* SS_FLAG_VALIDATE found an out-of-range index in a descriptor array    */
#define SS_ERR_TIMEOUT 6            /* a bounded device-side wait expired; the kernel drained and returned   */

/* ---- flags --------------------------------------------------------------------------------------------- */
#define SS_FLAG_VALIDATE 0x1u       /* check every index array on the device before it is used               */
#define SS_FLAG_FORCE_GENERIC 0x2u  /* attention: run every path through the simple one-row-per-warp kernel
                                       (no sharing, no tensor cores); a debugging aid and a second opinion  */
#define SS_FLAG_NO_TCGEN05 0x4u     /* attention: keep the plan but run shared-node / verification tiles on
                                       the simple kernel instead of the tcgen05 kernel                      */
#define SS_FLAG_WEAK_HASH 0x8u      /* dedup: truncate the path hash to 8 bits so that collisions are common;
                                       results must not change (tests the exact-comparison path)            */
#define SS_FLAG_TILES_2CTA 0x10u    /* attention: run the tcgen05 tile items on the kernel that keeps two CTAs
                                       per SM and works on 64-key tiles (default: the one-CTA-per-SM kernel with
                                       128-key tiles); same results within the accuracy contract             */

#define SS_MAX_DEPTH 16             /* maximum number of nodes on a root-to-leaf chain                       */

const char* ss_status_string(int32_t status);   /* host; static string, never NULL */

/* Reads the status word that the last call using this workspace recorded on the device.  Copies 4 bytes
 * device->host on `stream` and waits for that stream.  *out_status (host) receives SS_OK or an SS_ERR_*.
 * Returns SS_OK if the read itself worked. */
int32_t ss_last_device_status(const void* workspace, void* stream, int32_t* out_status);

/* =========================================================================================================
 * ss_dedup_paths - computation deduplication.
 *
 * Paper: Section "Computation Deduplication" - candidates whose input sequences are identical share one
 * forward pass; the number of logical candidates a sequence stands for is its "potential" size, and
 * sampled continuations are grouped by equality with one child per group whose potential is the group's
 * cardinality (worked example: three equal samples and one different -> potentials 3 and 1).
 *
 * Two logical paths i, j are duplicates iff ctx_key[i] == ctx_key[j] and their token-id sequences are equal
 * (same length, same ids).  Hashing is internal: collisions never change a result (equal-hash candidates are
 * compared token by token).
 *
 *   tok_ids        int32 [tok_offsets[n_paths]]   token ids, CSR by path
 *   tok_offsets    int64 [n_paths+1]              ascending, tok_offsets[0] may be any value >= 0
 *   ctx_key        int64 [n_paths] or NULL        opaque context that must also match (parent node, mode...)
 *   slot_in        int32 [n_paths] or NULL        KV slot (e.g. leaf node id) of each logical path
 *   n_paths        host, >= 0 (0: only *num_unique_out = 0 is written)
 *   flags          0 or SS_FLAG_WEAK_HASH
 *   canon_out          int32 [n_paths]   smallest index whose (ctx_key, sequence) equals path i's
 *   path_to_unique_out int32 [n_paths]   rank of canon_out[i] among the unique paths (ascending index order)
 *   unique_paths_out   int32 [n_paths]   first U entries valid: the unique paths, ascending
 *   multiplicity_out   int32 [n_paths]   first U entries valid: group sizes (the "potential" sizes)
 *   slot_out           int32 [n_paths] or NULL (must be NULL iff slot_in is NULL): slot_in[canon_out[i]]
 *   num_unique_out     int32 [1]         U
 *   workspace      >= ss_dedup_workspace_bytes(n_paths) bytes, 256-byte aligned
 *
 * Outputs are unique (no ordering freedom) and bit-exact with the plain std::map definition.
 * Errors: SS_ERR_INVALID_ARG, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_CUDA.
 * ======================================================================================================= */
int32_t ss_dedup_workspace_bytes(int32_t n_paths, size_t* out_bytes /* host */);
int32_t ss_dedup_paths(const int32_t* tok_ids, const int64_t* tok_offsets, const int64_t* ctx_key,
                       const int32_t* slot_in, int32_t n_paths, uint32_t flags, int32_t* canon_out,
                       int32_t* path_to_unique_out, int32_t* unique_paths_out, int32_t* multiplicity_out,
                       int32_t* slot_out, int32_t* num_unique_out, void* workspace, size_t workspace_bytes,
                       void* stream);

/* ss_gather_unique_paths - descriptor rows of the unique paths, in the layout ss_tree_attention takes.
 *
 * (Paper, Section "Computation Deduplication": a group of equal candidates gets ONE forward pass; this builds
 * the per-path arguments of that pass from the grouping.)  For p < U = *num_unique, with s = unique_paths[p]:
 *   u_leaf_out[p] = path_leaf_node[s],  u_q_len_out[p] = path_q_len[s],  u_q_src_out[p] = q_offsets[s]
 *   u_q_offsets_out[p+1] = u_q_len_out[0] + ... + u_q_len_out[p]          (u_q_offsets_out[0] = 0)
 * and for U <= p < n_paths: u_leaf_out[p] = -1, u_q_len_out[p] = 0, u_q_src_out[p] = 0,
 * u_q_offsets_out[p+1] = u_q_offsets_out[U].  Query rows are not moved: pass u_q_src_out as q_src_offsets.
 *
 *   unique_paths    int32 [n_paths]    device; first U entries used (ss_dedup_paths' unique_paths_out)
 *   num_unique      int32 [1]          device; U, clamped to [0, n_paths]
 *   n_paths         host, >= 0
 *   path_leaf_node  int32 [n_paths]    device; per LOGICAL path
 *   path_q_len      int32 [n_paths]    device
 *   q_offsets       int64 [n_paths+1]  device; row of each logical path's first query token
 *   u_leaf_out, u_q_len_out  int32 [n_paths];  u_q_offsets_out  int64 [n_paths+1];  u_q_src_out  int64 [n_paths]
 * No workspace, no host synchronisation; one launch on `stream`.  Errors: SS_ERR_INVALID_ARG, SS_ERR_CUDA. */
int32_t ss_gather_unique_paths(const int32_t* unique_paths, const int32_t* num_unique, int32_t n_paths,
                               const int32_t* path_leaf_node, const int32_t* path_q_len, const int64_t* q_offsets,
                               int32_t* u_leaf_out, int32_t* u_q_len_out, int64_t* u_q_offsets_out,
                               int64_t* u_q_src_out, void* stream);

/* ss_dedup_paths_static - ss_dedup_paths without a caller workspace and without any allocation.
 *
 * (The paper has no counterpart; this is a convenience of the library.)  It exists for callers that cannot ask
 * the CUDA allocator for scratch when they need a deduplication pass - for instance a serving engine whose free
 * HBM has all gone to its KV-cache pool, a scheduling loop that cannot afford the device-wide synchronisation an
 * allocation may imply, or an embedded plug-in that is not permitted to allocate.  The scratch is a fixed 2 MiB
 * array in device global memory that is part of the library image: every GPU that loads the library holds it
 * until the process exits.
 *
 *   Arguments and results are those of ss_dedup_paths (same meaning, same layout, bit-identical outputs), minus
 *   the workspace pair.  n_paths may be at most SS_DEDUP_STATIC_MAX_PATHS (65536); a larger value returns
 *   SS_ERR_UNSUPPORTED and nothing is launched - use ss_dedup_paths with your own workspace then.
 *   The call itself, and everything it calls, performs no cudaMalloc / cudaFree or other allocating routine.
 *   The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *   current); make that first call outside any stream capture.
 *   All calls on one device share the one array and the array keeps whatever the previous call left there (no
 *   part of it needs clearing between calls).  Two calls whose kernels can overlap on the GPU - different
 *   streams, or several host threads - race on it and give undefined results: serialise them.
 * Errors: as ss_dedup_paths, plus SS_ERR_UNSUPPORTED for n_paths above the maximum. */
#define SS_DEDUP_STATIC_MAX_PATHS 65536
int32_t ss_dedup_paths_static(const int32_t* tok_ids, const int64_t* tok_offsets, const int64_t* ctx_key,
                              const int32_t* slot_in, int32_t n_paths, uint32_t flags, int32_t* canon_out,
                              int32_t* path_to_unique_out, int32_t* unique_paths_out, int32_t* multiplicity_out,
                              int32_t* slot_out, int32_t* num_unique_out, void* stream);

/* =========================================================================================================
 * ss_tree_attention - attention over a tree of candidate paths that share KV prefixes.
 *
 * Paper: the serving substrate of Section "Experimental Setup" (paged attention, prefix KV caching and
 * sharing, fused attention kernels), used for the decode phase of expansion (Section "LLM Inference and
 * Serving") and for verification, which only prefills short steps (no decoding) (Section "Lazy
 * Verification").  The paper prints no formula; the operation is standard softmax attention:
 *
 *   for path p with KV sequence = concatenation of its nodes root -> leaf (length L), step length T:
 *     query token t (0 <= t < T), q head h, kv head g = h / (Hq/Hkv):
 *       s_j = sm_scale * <q[t,h,:], K[j,g,:]>            for keys j <= L - T + t  (bottom-right causal)
 *       out[t,h,:] = sum_j softmax(s)_j V[j,g,:]         lse[t,h] = ln sum_j exp(s_j)   (natural log)
 *     no visible key  =>  out = 0, lse = -inf.
 *
 * The step's own keys/values are expected to be in the pool already (they are the last T tokens of the
 * path's leaf node; appending them is outside this call).  Positional encoding is outside this call.
 *
 * Tree: nodes are numbered parents-before-children; node n holds node_kv_len[n] tokens in the pages
 * node_pages[node_page_offsets[n] .. node_page_offsets[n+1]) (16 tokens each; only the last page may be
 * partly filled; slots past the length are never read into a result).  A node that lies on the chain of
 * several paths is read once for all of them.  Paths are the UNIQUE paths (after ss_dedup_paths) in tree
 * order: the paths below any node are contiguous.  Every node with more than one path below it must hold a
 * multiple of 16 tokens.
 *
 * KV pool: bf16.  Element (page, kv head, token-in-page, dim) of K is
 *   k_pool[page*kv_page_stride + head*kv_head_stride + token*kv_token_stride + dim]   (strides in elements)
 * and likewise for v_pool.  Supported: kv_token_stride == head_dim (each (page, head) block is 16 contiguous
 * rows of 256 bytes), kv_page_stride and kv_head_stride multiples of 128 elements, k_pool and v_pool 256-byte
 * aligned.  The recommended pool is one allocation laid out [page][K|V][kv head][16][128].
 *
 * q   bf16 [total_q][Hq][128], rows of path p are q_offsets[p] .. q_offsets[p+1]-1 (or start at q_src_offsets[p] in
 *     a larger array, see the descriptor), 16-byte aligned
 * out bf16 [total_q][Hq][128]   (fp32 accumulation, rounded to nearest even), 32-byte aligned (the tile kernel
 *                               writes whole 32-byte sectors; any other alignment => SS_ERR_UNSUPPORTED)
 * lse fp32 [total_q][Hq]        or NULL
 *
 * Accuracy contract (inputs ~N(0,1) in bf16): |out - exact| <= 2e-2 max, 2e-3 mean; |lse - exact| <= 1e-3.
 *
 * Errors (host): SS_ERR_INVALID_ARG, SS_ERR_UNSUPPORTED, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_CUDA.
 * Errors (device, via ss_last_device_status): SS_ERR_UNSUPPORTED (depth, node length), SS_ERR_BAD_INPUT
 * (with SS_FLAG_VALIDATE), SS_ERR_WORKSPACE_TOO_SMALL (hints below were too low), SS_ERR_TIMEOUT.
 * ======================================================================================================= */
typedef struct ss_attn_desc {
  uint32_t struct_size;              /* = sizeof(ss_attn_desc_t) */
  uint32_t flags;                    /* SS_FLAG_* */
  int32_t num_q_heads, num_kv_heads; /* Hq % Hkv == 0 */
  int32_t head_dim, page_size;       /* 128, 16 */
  float sm_scale;                    /* 0 => 1/sqrt(head_dim) */
  int32_t max_sms;                   /* 0: use every SM; otherwise the tile and leaf kernels occupy at most this many.
                                        Their blocks are persistent and need an SM to themselves, so other streams'
                                        kernels wait for the whole call unless a few SMs are left out (the
                                        host-buffer step does that for the copy kernel of the step before it) */
  const void* k_pool;                /* bf16 */
  const void* v_pool;                /* bf16 */
  int64_t num_pages;                 /* pages addressable through k_pool / v_pool */
  int64_t kv_page_stride, kv_head_stride, kv_token_stride; /* elements */
  /* ---- tree ---- */
  int32_t num_nodes;
  int32_t reserved1;
  const int32_t* node_parent;        /* [num_nodes]  -1 for a root */
  const int32_t* node_kv_len;        /* [num_nodes]  >= 0 */
  const int64_t* node_page_offsets;  /* [num_nodes+1] */
  const int32_t* node_pages;         /* [total_node_pages] physical page ids */
  int64_t total_node_pages;          /* host copy of node_page_offsets[num_nodes] (an upper bound is fine) */
  /* ---- paths ---- */
  int32_t num_paths;                 /* capacity of the per-path arrays */
  int32_t reserved2;
  const int32_t* num_paths_dev;      /* NULL, or a device scalar <= num_paths holding the live path count
                                        (e.g. num_unique_out of ss_dedup_paths): no host sync needed between
                                        the two calls */
  const int32_t* path_leaf_node;     /* [num_paths] */
  const int32_t* path_q_len;         /* [num_paths] T >= 1 */
  const int64_t* q_offsets;          /* [num_paths+1] */
  int64_t total_q;                   /* host upper bound of q_offsets[live paths] */
  /* ---- sizing hints (host scalars; 0 = use the safe default; tight values shrink the workspace) ---- */
  int32_t max_depth;                 /* nodes on the longest chain; default SS_MAX_DEPTH */
  int32_t max_decode_paths;          /* paths with T == 1; default num_paths */
  /* ---- optional query indirection ---- */
  const int64_t* q_src_offsets;      /* NULL, or [num_paths]: row of q where path p's T query rows start (default
                                        q_offsets[p]).  Lets the caller leave q in logical-candidate order after
                                        ss_dedup_paths instead of gathering the unique paths' rows; out / lse rows
                                        stay at q_offsets[p] */
  int64_t q_src_rows;                /* rows addressable through q when q_src_offsets is given (host) */
  /* ---- data ---- */
  const void* q;
  void* out;
  float* lse;
} ss_attn_desc_t;

int32_t ss_tree_attention_workspace_bytes(const ss_attn_desc_t* desc /* host */, size_t* out_bytes /* host */);
int32_t ss_tree_attention(const ss_attn_desc_t* desc /* host */, void* workspace, size_t workspace_bytes,
                          void* stream);

/* =========================================================================================================
 * ss_topk_prune - keep the k best-scored candidates of every problem.
 *
 * Paper: Section "Early Pruning of Search Tree" - a candidate whose score ranks below the top-k cannot be
 * part of the final top-k and is pruned; Section "Test-Time Scaling" - top-k = N / M (beam size / width).
 * Ordering: score descending, ties to the lower index (the paper cannot distinguish equal scores); -0.0 equals
 * +0.0; NaN ranks below every number.  The result is unique.
 *
 *   scores        fp32 [n_total]
 *   seg_offsets   int32 [n_segments+1]  ascending; segment s = candidates seg_offsets[s] .. seg_offsets[s+1]-1
 *   n_segments    host >= 0;  n_total host >= seg_offsets[n_segments];  k host >= 1
 *   survivors_out int32 [n_segments][k]  global candidate indices, best first, -1 padded when a segment has
 *                 fewer than k candidates
 *   keep_out      uint8 [n_total]        1 iff the candidate survives (entries outside every segment: 0)
 *   workspace     >= ss_topk_workspace_bytes(n_total) bytes, 256-byte aligned
 * Errors: SS_ERR_INVALID_ARG, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_CUDA (host); SS_ERR_BAD_INPUT via
 * ss_last_device_status(workspace) if a segment does not lie inside [0, n_total] (it is then treated as empty).
 * ======================================================================================================= */
int32_t ss_topk_workspace_bytes(int32_t n_total, size_t* out_bytes /* host */);
int32_t ss_topk_prune(const float* scores, const int32_t* seg_offsets, int32_t n_segments, int32_t n_total,
                      int32_t k, int32_t* survivors_out, uint8_t* keep_out, void* workspace,
                      size_t workspace_bytes, void* stream);

/* =========================================================================================================
 * ss_early_prune - pruning while only part of a problem's candidates has been verified.
 *
 * Paper: Section "Early Pruning of Search Tree".  Rule 1: once more than k candidates are verified, a verified
 * candidate ranked below the k best verified ones can no longer reach the final top-k and is pruned.  Rule 2: PRM
 * scores lie in [0, 1]; once k verified candidates have the perfect score (>= 1.0) they are final - the first k of
 * them by index are selected and every other candidate of the problem, verified or not, is pruned.  Worked example
 * of the paper (k = 1): B verified -> continues; D verified with a lower score -> pruned; C perfect -> A, B, D
 * pruned, C selected.  Ordering and special values as in ss_topk_prune.
 *
 *   scores        fp32 [n_total]    only entries with verified[i] != 0 are read
 *   verified      uint8 [n_total]
 *   seg_offsets   int32 [n_segments+1]; k host >= 1
 *   pruned_out    uint8 [n_total]   1 iff the candidate must stop (entries outside every segment: 0)
 *   selected_out  int32 [n_segments][k]  the selection of a FINAL segment (best first / perfect ones by index),
 *                 -1 padded; all -1 while the segment is not final
 *   final_out     uint8 [n_segments] 1 iff rule 2 fired or every candidate of the segment is verified (then
 *                 selected_out equals the survivors of ss_topk_prune)
 *   workspace     >= ss_topk_workspace_bytes(n_total) bytes, 256-byte aligned
 * Errors: SS_ERR_INVALID_ARG, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_CUDA (host); SS_ERR_BAD_INPUT via
 * ss_last_device_status(workspace) if a segment does not lie inside [0, n_total] (it is then treated as empty).
 * ======================================================================================================= */
int32_t ss_early_prune(const float* scores, const uint8_t* verified, const int32_t* seg_offsets, int32_t n_segments,
                       int32_t n_total, int32_t k, uint8_t* pruned_out, int32_t* selected_out, uint8_t* final_out,
                       void* workspace, size_t workspace_bytes, void* stream);

/* =========================================================================================================
 * ss_branch_sample - the draws of on-demand branching.
 *
 * Paper: Section "Computation Deduplication" - a sequence with potential size n runs one forward pass and then
 * draws n next tokens independently from that one distribution; equal samples are grouped and every
 * group becomes one child sequence whose potential size is the group's cardinality.  This call does the sampling;
 * the grouping is ss_dedup_paths on the (sequence, token) pairs it returns (tok_ids = tokens_out with one token per
 * path, ctx_key = seq_out): multiplicity_out are then the children's potential sizes.  (The paper batches the
 * sampler by potential size because its sampler needs one output shape per call; one launch handles any mix here.)
 *
 * Distribution: softmax(logits / temperature).  The random numbers are inputs.  Rule (evaluated in fp64):
 *   e_v = exp((logit_v - max) / temperature), C_v = e_0 + .. + e_v, token = the smallest v with C_v > u * C_{V-1}.
 *
 *   logits        fp32 [n_seq][vocab]   (-inf allowed: probability 0; at least one finite value per row)
 *   draw_offsets  int64 [n_seq+1]       draws of sequence s are draw_offsets[s] .. draw_offsets[s+1]-1
 *                                       (draw_offsets[s+1] - draw_offsets[s] = its potential size)
 *   uniforms      fp32 [draw_offsets[n_seq]]  in [0, 1)
 *   n_seq, vocab  host;  temperature host > 0;  vocab <= 2097152 (else SS_ERR_UNSUPPORTED)
 *   tokens_out    int32 [draws]   sampled token of every draw
 *   seq_out       int64 [draws]   the sequence every draw belongs to
 * Errors: SS_ERR_INVALID_ARG, SS_ERR_UNSUPPORTED, SS_ERR_CUDA.
 * ======================================================================================================= */
int32_t ss_branch_sample(const float* logits, const int64_t* draw_offsets, const float* uniforms, int32_t n_seq,
                         int32_t vocab, float temperature, int32_t* tokens_out, int64_t* seq_out, void* stream);

/* =========================================================================================================
 * ss_build_prefix_tree - radix tree of candidate paths over whole KV pages, from raw token ids.
 *
 * Paper: Section "Computation Deduplication" (a quarter to a half of the tokens that the candidates of a step
 * generate are common across candidates) and Section "Experimental Setup" (prefix KV caching and sharing):
 * beyond removing candidates that are equal as a whole (ss_dedup_paths), candidates that agree on a prefix can keep
 * that prefix's KV once.  This call finds the sharing: it returns the tree (parents before children) in exactly the
 * form ss_tree_attention takes, with only WHOLE pages shared, so that a node's pages can be the physical pages of
 * any path below it.
 *
 * Definition (unique): paths are ordered by token sequence (a proper prefix first, then the input index).  A group
 * of at least two neighbouring paths that share more full pages than the chain above them holds gets an inner node
 * with exactly the pages all of them share; the group splits where two neighbours share no further page; a single
 * path gets a private leaf node with whatever the chain above it does not hold (possibly nothing).  Nodes are
 * numbered depth-first along the order, so the paths below a node are contiguous.
 *
 *   tok_ids, tok_offsets  as in ss_dedup_paths, with tok_offsets[0] == 0
 *   n_paths               host, 0 .. SS_PREFIX_TREE_MAX_PATHS;  total_tok  host, >= tok_offsets[n_paths]
 *   page_size             host, >= 1 (16 for ss_tree_attention)
 *   order_out           int32 [n_paths]     input index of the path of every rank
 *   path_leaf_node_out  int32 [n_paths]     by rank
 *   node_parent_out, node_kv_len_out                int32 [2*n_paths]   first *num_nodes_out entries valid
 *   node_src_path_out, node_src_offset_out          int32 [2*n_paths]   an input path that contains the node's tokens
 *                                                                        and the position where they start in it
 *   num_nodes_out       int32 [1]           n_paths leaves + the inner nodes (0 after a device-side error)
 *   workspace           >= ss_prefix_tree_workspace_bytes(...) bytes, 256-byte aligned; its first word is the device
 *                       status (ss_last_device_status): SS_ERR_BAD_INPUT if the internal 64-bit page hashes collided
 *                       in a way that mis-ordered two paths (the tree is then withheld, never wrong)
 * Errors (host): SS_ERR_INVALID_ARG, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_CUDA.
 * ======================================================================================================= */
#define SS_PREFIX_TREE_MAX_PATHS (1 << 20)
int32_t ss_prefix_tree_workspace_bytes(int32_t n_paths, int64_t total_tok, int32_t page_size,
                                       size_t* out_bytes /* host */);
int32_t ss_build_prefix_tree(const int32_t* tok_ids, const int64_t* tok_offsets, int32_t n_paths, int64_t total_tok,
                             int32_t page_size, int32_t* order_out, int32_t* path_leaf_node_out,
                             int32_t* node_parent_out, int32_t* node_kv_len_out, int32_t* node_src_path_out,
                             int32_t* node_src_offset_out, int32_t* num_nodes_out, void* workspace,
                             size_t workspace_bytes, void* stream);

/* =========================================================================================================
 * ss_candidate_step_host - one pass of the whole path for per-step data that lives in HOST memory.
 *
 * Paper: the system overview figure and Sections "Computation Deduplication", "Lazy Verification" and "Early
 * Pruning of Search Tree" - per expansion / verification step the candidates are deduplicated, the unique ones get one attention pass over the
 * shared KV prefixes, and the scored candidates are pruned to the top-k.  This call is that sequence for a caller
 * whose candidates, query activations and scores are produced on the host side of the bus:
 *   asynchronous copies host -> device of every per-step input  ->  ss_dedup_paths  ->  ss_gather_unique_paths  ->
 *   ss_tree_attention (queries read in place through the gathered offsets)  ->  ss_topk_prune  ->
 *   asynchronous copies device -> host of every result.
 * With SS_STEP_COMPACT_TRANSFERS in `flags`, and out / lse page-locked AND mapped into the device's address space
 * (memory from cudaHostAlloc / cudaHostRegister), only the live rows of out / lse come back - the first
 * u_q_offsets[num_unique]: a duplicate candidate gets no forward pass, hence no output of its own - written by a small
 * kernel straight into the host buffers; the rest of out / lse is left untouched.  (Buffers the device cannot address
 * are returned whole, as without the flag.)
 * Everything is enqueued on `stream`; the call does not synchronise, and it allocates nothing: staging buffers,
 * results and the workspaces of the three calls are carved out of `device_arena` (caller-owned, 256-byte aligned,
 * >= ss_candidate_step_host_arena_bytes).  The KV pool and the tree stay resident on the device: they are the
 * cache state of the method, described by the resident fields of `attn` (flags, heads, sm_scale, pool, strides,
 * tree arrays, total_node_pages, max_depth, max_decode_paths); the path, query and output fields of `attn` are
 * ignored.  Host buffers should be page-locked, else the copies are synchronous (results are the same).  A caller
 * that alternates between two or three (arena, stream, host buffer) sets overlaps the copies of one step with the
 * kernels of another.  Results are valid once `stream` has drained; *device_status then holds what
 * ss_last_device_status would report for the attention call.
 *
 * Inputs (host): as the arguments of the same name of ss_dedup_paths, ss_gather_unique_paths, ss_tree_attention
 * (q: bf16 [total_q][Hq][128] in logical-candidate order) and ss_topk_prune.  ctx_key may be NULL; slot_in and
 * slot_out must both be given or both be NULL; lse may be NULL.
 * Results (host): canon, path_to_unique, unique_paths, multiplicity, slot_out [n_paths], num_unique [1],
 * u_q_offsets int64 [n_paths+1] (rows of out / lse of unique path p: u_q_offsets[p] .. u_q_offsets[p+1]-1),
 * out bf16 [total_q][Hq][128], lse fp32 [total_q][Hq], survivors int32 [n_segments][top_k], keep uint8 [n_paths],
 * device_status int32 [1].
 * Errors: SS_ERR_INVALID_ARG, SS_ERR_WORKSPACE_TOO_SMALL, SS_ERR_UNSUPPORTED, SS_ERR_CUDA (host); the device-side
 * errors of ss_tree_attention arrive in *device_status.
 * ======================================================================================================= */
#define SS_STEP_COMPACT_TRANSFERS 0x1u   /* return only the live rows of out / lse (needs them mapped, see above) */
typedef struct ss_host_step {
  uint32_t struct_size;              /* = sizeof(ss_host_step_t) */
  uint32_t dedup_flags;              /* 0 or SS_FLAG_WEAK_HASH */
  const ss_attn_desc_t* attn;        /* host; resident fields only (see above) */
  int32_t n_paths, n_segments, top_k;
  uint32_t flags;                    /* 0 or SS_STEP_COMPACT_TRANSFERS */
  int64_t total_tok;                 /* = tok_offsets[n_paths] - tok_offsets[0], and tok_offsets[0] must be 0 */
  int64_t total_q;                   /* = q_offsets[n_paths], and q_offsets[0] must be 0 */
  /* per-step inputs, host memory */
  const int32_t* tok_ids;
  const int64_t* tok_offsets;
  const int64_t* ctx_key;
  const int32_t* slot_in;
  const int32_t* path_leaf_node;
  const int32_t* path_q_len;
  const int64_t* q_offsets;
  const void* q;
  const float* scores;
  const int32_t* seg_offsets;
  /* results, host memory */
  int32_t* canon;
  int32_t* path_to_unique;
  int32_t* unique_paths;
  int32_t* multiplicity;
  int32_t* slot_out;
  int32_t* num_unique;
  int64_t* u_q_offsets;
  void* out;
  float* lse;
  int32_t* survivors;
  uint8_t* keep;
  int32_t* device_status;
} ss_host_step_t;

int32_t ss_candidate_step_host_arena_bytes(const ss_host_step_t* step /* host */, size_t* out_bytes /* host */);
int32_t ss_candidate_step_host(const ss_host_step_t* step /* host */, void* device_arena, size_t arena_bytes,
                               void* stream);

/* =========================================================================================================
 * Diagnostics
 * ======================================================================================================= */
/* Number of kernels this library has launched in this process since it was loaded (host counter). */
int64_t ss_launch_count(void);

/* Per-phase timing of ss_tree_attention with CUDA events (diagnostics; no paper counterpart).
 * While enabled, every ss_tree_attention call records events on its stream around each phase
 * (SS_PHASE_*); the events come from a fixed pool created on first use (calls beyond the pool are not timed).
 * ss_profile_read waits for the recorded events, adds up the milliseconds and the number of timed calls per
 * phase into the host arrays (each SS_NUM_PHASES long; either may be NULL) and clears the record.
 * Not thread-safe; meant for a benchmark harness. */
#define SS_PHASE_PLAN 0
#define SS_PHASE_TILES 1      /* tcgen05 tile items: shared-node (stacked decode rows) and verification tiles */
#define SS_PHASE_LEAVES 2     /* bandwidth-bound decode-leaf items */
#define SS_PHASE_GENERIC 3
#define SS_PHASE_MERGE 4
#define SS_NUM_PHASES 5
int32_t ss_profile_enable(int32_t on);
int32_t ss_profile_read(float* phase_ms /* host */, int64_t* phase_calls /* host */);

/* CTAs of the tcgen05 tile kernel that fit one SM according to the CUDA occupancy query (0 before the first
 * ss_tree_attention call that used the kernel).  Diagnostics; no paper counterpart. */
int32_t ss_debug_tile_kernel_occupancy(void);

/* One 128 x N x K bf16 tile product on the tcgen05 tensor cores, C[128][N] (fp32, row-major) = A[128][K] *
 * op(B), with the same shared-memory descriptors and TMEM read-out as the attention kernel.
 *   b_is_mn_major == 0: B is [N][K] row-major (the K-operand form, like keys);  C = A * B^T
 *   b_is_mn_major == 1: B is [K][N] row-major (the value form);                 C = A * B
 * N in {64, 128}, K a multiple of 64 and <= 256.  No paper counterpart: a self-test of the tensor-core
 * plumbing.  status_out: device int32[1], receives SS_OK or SS_ERR_TIMEOUT. */
int32_t ss_debug_umma_tile(const void* a_bf16, const void* b_bf16, float* c, int32_t n, int32_t k,
                           int32_t b_is_mn_major, int32_t* status_out, void* stream);

/* Self-test of the bounded wait every kernel role uses (no paper counterpart): one CTA waits on a shared-memory
 * barrier that nothing ever completes.  The wait must give up after its time limit (about 0.2 s), raise the CTA's
 * abort flag and return, and the kernel must then end normally.  status_out: device int32[2];
 * status_out[0] receives SS_ERR_TIMEOUT when that happened (SS_OK if the wait claimed success, which would be a bug),
 * status_out[1] the clocks the wait took, in millions.  Returns SS_OK when the kernel was launched. */
int32_t ss_debug_bounded_wait(int32_t* status_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECSCALE_H_ */
