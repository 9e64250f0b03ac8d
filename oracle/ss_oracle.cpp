// CPU oracle for the candidate-path hot path of speculative expand-verify-select search.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of what the CUDA
// library must compute.  It shares no code, header, table or helper with the CUDA path and must never be
// called from it; only the test-suite, the smoke check and the benchmark's cpu_baseline / reference arm may
// load it.  Everything is host memory; floating point is fp64.
//
//   ss_oracle_dedup           Computation deduplication: candidates whose input sequences are identical form one
//                             group that is computed once; the group's size is the sequence's "potential"
//                             (paper, Section "Computation Deduplication").  Plain definition with std::map.
//   ss_oracle_tree_attention  Softmax attention of every candidate path over its own root-to-leaf KV
//                             sequence (paper: attention over paged KV with shared prefixes, Sections
//                             "LLM Inference and Serving" and "Experimental Setup").  The paper prints no
//                             formula; this is the textbook definition, written per path with the path's
//                             whole K/V materialised contiguously - no tiling, no sharing, no merging.
//   ss_oracle_early_prune     The same selection while only part of the candidates is verified: rule 1 (ranked
//                             below the top-k of the verified ones => pruned) and rule 2 (k perfect scores =>
//                             final), paper, Section "Early Pruning of Search Tree".
//   ss_oracle_branch_sample   On-demand branching: the potential-many next-token draws of a sequence from one
//                             logits row (paper, Section "Computation Deduplication"); inverse-CDF sampling with
//                             the uniform random numbers passed in.
//   ss_oracle_topk            Selection of the top-k candidates by score (paper, Section "Early Pruning of
//                             Search Tree": a candidate ranked below the top-k cannot be selected;
//                             top-k = N / M).  Plain stable sort.
//
// Readings where the paper is silent are listed in the design notes of the repository; the ones this file
// fixes: scale given by the caller; natural-log LSE; q head h reads kv head h / (Hq/Hkv); bottom-right
// causal alignment (query t of a T-token step sees keys 0 .. L-T+t); an empty key set gives out = 0,
// lse = -inf; ties in top-k go to the lower index; -0.0 == +0.0; NaN ranks below every number.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <map>
#include <thread>
#include <utility>
#include <vector>

namespace {

inline double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}

}  // namespace

extern "C" {

// ---------------------------------------------------------------------------------------------------------
// Dedup.  key = (ctx_key[i], token-id vector of path i).  canon[i] = first index holding the same key;
// unique list = ascending indices with canon[i] == i; path_to_unique[i] = rank of canon[i] in that list;
// multiplicity[u] = size of the group of unique path u; slot_out[i] = slot_in[canon[i]].
// ctx_key / slot_in / slot_out may be null.  Returns the number of unique paths.
// ---------------------------------------------------------------------------------------------------------
int32_t ss_oracle_dedup(const int32_t* tok_ids, const int64_t* tok_offsets, const int64_t* ctx_key,
                        const int32_t* slot_in, int32_t n_paths, int32_t* canon, int32_t* path_to_unique,
                        int32_t* unique_paths, int32_t* multiplicity, int32_t* slot_out) {
  typedef std::pair<int64_t, std::vector<int32_t> > Key;
  std::map<Key, int32_t> first;
  for (int32_t i = 0; i < n_paths; ++i) {
    Key key(ctx_key ? ctx_key[i] : 0,
            std::vector<int32_t>(tok_ids + tok_offsets[i], tok_ids + tok_offsets[i + 1]));
    std::map<Key, int32_t>::iterator it = first.find(key);
    if (it == first.end()) {
      first.insert(std::make_pair(key, i));
      canon[i] = i;
    } else {
      canon[i] = it->second;
    }
  }
  int32_t u = 0;
  std::vector<int32_t> rank(n_paths > 0 ? n_paths : 1, -1);
  for (int32_t i = 0; i < n_paths; ++i) {
    if (canon[i] == i) {
      rank[i] = u;
      unique_paths[u] = i;
      multiplicity[u] = 0;
      ++u;
    }
  }
  for (int32_t i = 0; i < n_paths; ++i) {
    path_to_unique[i] = rank[canon[i]];
    multiplicity[rank[canon[i]]] += 1;
    if (slot_in && slot_out) slot_out[i] = slot_in[canon[i]];
  }
  return u;
}

// ---------------------------------------------------------------------------------------------------------
// Attention.  For each path p: walk root -> leaf, copy each node's tokens out of the paged pool into
// K_p[L][Hkv][D], V_p[L][Hkv][D] (fp64).  For each query token t < T_p and q head h (kv head g = h / G):
//   s_j = sm_scale * sum_d q[t,h,d] K_p[j,g,d]   for j <= L - T_p + t
//   m = max_j s_j,  Z = sum_j exp(s_j - m),  out[t,h,:] = sum_j exp(s_j - m)/Z * V_p[j,g,:],  lse = m + ln Z
// Pool element (page, head, token-in-page, d) of K is k_pool[page*page_stride + head*head_stride +
// token*token_stride + d]; same for v_pool.  q is bf16 bits [total_q][Hq][D]; out fp64 same shape;
// lse fp64 [total_q][Hq].  Paths are independent and are spread over n_threads.
// Returns 0, or -1 on a malformed tree (a parent index >= its child, a chain deeper than the node count).
// ---------------------------------------------------------------------------------------------------------
struct AttnArgs {
  int Hq, Hkv, D, page_size;
  double sm_scale;
  const uint16_t *k_pool, *v_pool;
  int64_t page_stride, head_stride, token_stride;
  int32_t num_nodes;
  const int32_t *node_parent, *node_kv_len;
  const int64_t* node_page_offsets;
  const int32_t* node_pages;
  int32_t num_paths;
  const int32_t *path_leaf_node, *path_q_len;
  const int64_t* q_offsets;
  const uint16_t* q;
  double *out, *lse;
};

static void attend_one_path(const AttnArgs& a, int32_t p) {
  const int G = a.Hq / a.Hkv;
  // chain root -> leaf
  std::vector<int32_t> chain;
  for (int32_t n = a.path_leaf_node[p]; n >= 0; n = a.node_parent[n]) chain.push_back(n);
  std::reverse(chain.begin(), chain.end());
  int64_t L = 0;
  for (size_t c = 0; c < chain.size(); ++c) L += a.node_kv_len[chain[c]];
  std::vector<double> K(static_cast<size_t>(L) * a.Hkv * a.D), V(K.size());
  int64_t pos = 0;
  for (size_t c = 0; c < chain.size(); ++c) {
    const int32_t n = chain[c];
    for (int32_t j = 0; j < a.node_kv_len[n]; ++j, ++pos) {
      const int64_t page = a.node_pages[a.node_page_offsets[n] + j / a.page_size];
      const int64_t in_page = j % a.page_size;
      for (int g = 0; g < a.Hkv; ++g) {
        const int64_t src = page * a.page_stride + g * a.head_stride + in_page * a.token_stride;
        double* kd = &K[(static_cast<size_t>(pos) * a.Hkv + g) * a.D];
        double* vd = &V[(static_cast<size_t>(pos) * a.Hkv + g) * a.D];
        for (int d = 0; d < a.D; ++d) {
          kd[d] = bf16_to_double(a.k_pool[src + d]);
          vd[d] = bf16_to_double(a.v_pool[src + d]);
        }
      }
    }
  }
  const int32_t T = a.path_q_len[p];
  std::vector<double> s(static_cast<size_t>(L > 0 ? L : 1)), qrow(a.D), acc(a.D);
  for (int32_t t = 0; t < T; ++t) {
    const int64_t row = a.q_offsets[p] + t;
    const int64_t visible = L - T + t + 1;  // keys 0 .. L-T+t
    for (int h = 0; h < a.Hq; ++h) {
      const int g = h / G;
      double* o = a.out + (row * a.Hq + h) * a.D;
      double* l = a.lse + row * a.Hq + h;
      for (int d = 0; d < a.D; ++d) qrow[d] = bf16_to_double(a.q[(row * a.Hq + h) * a.D + d]);
      if (visible <= 0) {
        for (int d = 0; d < a.D; ++d) o[d] = 0.0;
        *l = -std::numeric_limits<double>::infinity();
        continue;
      }
      double m = -std::numeric_limits<double>::infinity();
      for (int64_t j = 0; j < visible; ++j) {
        const double* kd = &K[(static_cast<size_t>(j) * a.Hkv + g) * a.D];
        double dot = 0.0;
        for (int d = 0; d < a.D; ++d) dot += qrow[d] * kd[d];
        s[j] = a.sm_scale * dot;
        if (s[j] > m) m = s[j];
      }
      double Z = 0.0;
      for (int d = 0; d < a.D; ++d) acc[d] = 0.0;
      for (int64_t j = 0; j < visible; ++j) {
        const double w = std::exp(s[j] - m);
        Z += w;
        const double* vd = &V[(static_cast<size_t>(j) * a.Hkv + g) * a.D];
        for (int d = 0; d < a.D; ++d) acc[d] += w * vd[d];
      }
      for (int d = 0; d < a.D; ++d) o[d] = acc[d] / Z;
      *l = m + std::log(Z);
    }
  }
}

int32_t ss_oracle_tree_attention(int32_t Hq, int32_t Hkv, int32_t D, int32_t page_size, double sm_scale,
                                 const uint16_t* k_pool, const uint16_t* v_pool, int64_t page_stride,
                                 int64_t head_stride, int64_t token_stride, int32_t num_nodes,
                                 const int32_t* node_parent, const int32_t* node_kv_len,
                                 const int64_t* node_page_offsets, const int32_t* node_pages,
                                 int32_t num_paths, const int32_t* path_leaf_node, const int32_t* path_q_len,
                                 const int64_t* q_offsets, const uint16_t* q, double* out, double* lse,
                                 int32_t n_threads) {
  for (int32_t n = 0; n < num_nodes; ++n)
    if (node_parent[n] >= n || node_parent[n] < -1) return -1;
  for (int32_t p = 0; p < num_paths; ++p)
    if (path_leaf_node[p] < 0 || path_leaf_node[p] >= num_nodes) return -1;
  AttnArgs a;
  a.Hq = Hq; a.Hkv = Hkv; a.D = D; a.page_size = page_size; a.sm_scale = sm_scale;
  a.k_pool = k_pool; a.v_pool = v_pool;
  a.page_stride = page_stride; a.head_stride = head_stride; a.token_stride = token_stride;
  a.num_nodes = num_nodes; a.node_parent = node_parent; a.node_kv_len = node_kv_len;
  a.node_page_offsets = node_page_offsets; a.node_pages = node_pages;
  a.num_paths = num_paths; a.path_leaf_node = path_leaf_node; a.path_q_len = path_q_len;
  a.q_offsets = q_offsets; a.q = q; a.out = out; a.lse = lse;
  if (n_threads < 1) n_threads = 1;
  if (n_threads == 1 || num_paths < 2) {
    for (int32_t p = 0; p < num_paths; ++p) attend_one_path(a, p);
    return 0;
  }
  std::vector<std::thread> pool;
  for (int32_t w = 0; w < n_threads; ++w)
    pool.push_back(std::thread([&a, w, n_threads]() {
      for (int32_t p = w; p < a.num_paths; p += n_threads) attend_one_path(a, p);
    }));
  for (size_t w = 0; w < pool.size(); ++w) pool[w].join();
  return 0;
}

// ---------------------------------------------------------------------------------------------------------
// Top-k.  Per segment [seg_offsets[s], seg_offsets[s+1]): stable sort of the indices by score descending
// (stable => lower index first among equal scores; NaN last, NaNs among themselves by index); survivors =
// the first min(k, n) GLOBAL indices in that order, padded with -1 to k; keep[i] = 1 iff i survives.
// ---------------------------------------------------------------------------------------------------------
static bool score_before(float a, float b) {  // strict "a ranks before b" ignoring the index
  const bool an = std::isnan(a), bn = std::isnan(b);
  if (an || bn) return !an && bn;
  return a > b;  // -0.0 > +0.0 is false both ways: equal
}

void ss_oracle_topk(const float* scores, const int32_t* seg_offsets, int32_t n_segments, int32_t k,
                    int32_t* survivors, uint8_t* keep) {
  for (int32_t s = 0; s < n_segments; ++s) {
    const int32_t lo = seg_offsets[s], hi = seg_offsets[s + 1];
    std::vector<int32_t> idx;
    for (int32_t i = lo; i < hi; ++i) {
      idx.push_back(i);
      keep[i] = 0;
    }
    std::stable_sort(idx.begin(), idx.end(),
                     [scores](int32_t x, int32_t y) { return score_before(scores[x], scores[y]); });
    for (int32_t j = 0; j < k; ++j) {
      if (j < static_cast<int32_t>(idx.size())) {
        survivors[static_cast<int64_t>(s) * k + j] = idx[j];
        keep[idx[j]] = 1;
      } else {
        survivors[static_cast<int64_t>(s) * k + j] = -1;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Early pruning during speculation (paper, Section "Early Pruning of Search Tree").  Only part of a problem's
// candidates has been verified so far (verified[i] != 0; the scores of the others are ignored).  Per segment:
//   rule 2  if at least k verified candidates have the perfect score (>= 1.0): the first k of them by index are
//           selected, the segment is final, and every other candidate - verified or not - is pruned;
//   rule 1  otherwise, if more than k candidates are verified: a verified candidate that ranks below the k best
//           verified ones (score descending, lower index first among equals) cannot reach the final top-k and is
//           pruned; unverified candidates keep running;
//   if every candidate of the segment is verified the segment is final as well and the selection is the plain
//   top-k.
// pruned[i] = 1 iff candidate i must stop; selected = [P][k] indices (-1 padded; all -1 unless final);
// final_out[s] = 1 iff segment s is final.
// ---------------------------------------------------------------------------------------------------------
void ss_oracle_early_prune(const float* scores, const uint8_t* verified, const int32_t* seg_offsets,
                           int32_t n_segments, int32_t k, uint8_t* pruned, int32_t* selected, uint8_t* final_out) {
  for (int32_t s = 0; s < n_segments; ++s) {
    const int32_t lo = seg_offsets[s], hi = seg_offsets[s + 1];
    for (int32_t j = 0; j < k; ++j) selected[static_cast<int64_t>(s) * k + j] = -1;
    for (int32_t i = lo; i < hi; ++i) pruned[i] = 0;
    final_out[s] = 0;
    std::vector<int32_t> ver, perfect;
    for (int32_t i = lo; i < hi; ++i) {
      if (!verified[i]) continue;
      ver.push_back(i);
      if (scores[i] >= 1.0f) perfect.push_back(i);
    }
    if (static_cast<int32_t>(perfect.size()) >= k) {
      for (int32_t i = lo; i < hi; ++i) pruned[i] = 1;
      for (int32_t j = 0; j < k; ++j) {
        selected[static_cast<int64_t>(s) * k + j] = perfect[j];
        pruned[perfect[j]] = 0;
      }
      final_out[s] = 1;
      continue;
    }
    std::stable_sort(ver.begin(), ver.end(),
                     [scores](int32_t x, int32_t y) { return score_before(scores[x], scores[y]); });
    const bool all_verified = static_cast<int32_t>(ver.size()) == hi - lo;
    if (static_cast<int32_t>(ver.size()) > k)
      for (size_t r = k; r < ver.size(); ++r) pruned[ver[r]] = 1;
    if (all_verified) {
      final_out[s] = 1;
      for (int32_t j = 0; j < k && j < static_cast<int32_t>(ver.size()); ++j)
        selected[static_cast<int64_t>(s) * k + j] = ver[j];
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// On-demand branching, sampling half (paper, Section "Computation Deduplication"): a sequence whose potential
// size is n runs ONE forward pass and then draws n next tokens "as independent trials from the same
// distribution"; equal draws are grouped afterwards (ss_oracle_dedup on (sequence, token) pairs gives the groups
// and their cardinalities = the children's potential sizes).
// Distribution: softmax(logits / temperature) over the vocabulary.  The random numbers are INPUTS: draw k of
// sequence s uses uniforms[draw_offsets[s] + k] in [0, 1).  Inverse-CDF rule in fp64:
//   e_v = exp((logit_v - max) / temperature),  C_v = e_0 + ... + e_v,  Z = C_{V-1},
//   token = the smallest v with C_v > u * Z.
// tokens_out[d] = sampled token of draw d, seq_out[d] = its sequence.  margin_out (may be null) receives, per
// draw, min(|u*Z - C_{token-1}|, |C_token - u*Z|) / Z: how far the draw is from flipping to a neighbouring token.
// ---------------------------------------------------------------------------------------------------------
void ss_oracle_branch_sample(const float* logits, const int64_t* draw_offsets, const float* uniforms,
                             int32_t n_seq, int32_t vocab, double temperature, int32_t* tokens_out,
                             int64_t* seq_out, double* margin_out) {
  std::vector<double> cdf(static_cast<size_t>(vocab > 0 ? vocab : 1));
  for (int32_t s = 0; s < n_seq; ++s) {
    const float* row = logits + static_cast<int64_t>(s) * vocab;
    double mx = -std::numeric_limits<double>::infinity();
    for (int32_t v = 0; v < vocab; ++v) mx = std::max(mx, static_cast<double>(row[v]));
    double run = 0.0;
    for (int32_t v = 0; v < vocab; ++v) {
      run += std::exp((static_cast<double>(row[v]) - mx) / temperature);
      cdf[v] = run;
    }
    const double Z = run;
    for (int64_t d = draw_offsets[s]; d < draw_offsets[s + 1]; ++d) {
      const double target = static_cast<double>(uniforms[d]) * Z;
      int32_t tok = vocab - 1;
      for (int32_t v = 0; v < vocab; ++v)
        if (cdf[v] > target) { tok = v; break; }
      tokens_out[d] = tok;
      seq_out[d] = s;
      if (margin_out) {
        const double below = tok > 0 ? cdf[tok - 1] : 0.0;
        margin_out[d] = std::min(std::fabs(target - below), std::fabs(cdf[tok] - target)) / Z;
      }
    }
  }
}

}  // extern "C"
