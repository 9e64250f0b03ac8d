"""Seeded synthetic candidate-path trees (inputs only; none of the method's arithmetic lives here).

The paper evaluates on math-reasoning datasets with real generator / reward models.  Those are not
available, so every input is a seeded stand-in that keeps the *structure* of the workload: P concurrent
problems, N candidate paths per problem that share the prompt prefix, per-candidate suffixes of diverging
length, a fraction of identical candidates (computation deduplication, Section "Computation
Deduplication"), and verification steps of 16-128 tokens (Section "Lazy Verification").

This module is shared by the CPU oracle's tests and by the CUDA path's tests/bench.  It produces

  * the tree (nodes, parents, page lists), in DFS order so that every node's descendant paths are contiguous,
  * the logical candidate list (leaf node, step length T, token ids, context key, KV slot),
  * bulk tensors (paged bf16 KV pool, bf16 queries, fp32 scores), filled with a torch generator on the
    requested device (host for small cases, the GPU for the 42 GB case).

Nothing here hashes, sorts, de-duplicates, attends or selects.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

VOCAB = 151936          # token ids are uniform in [0, VOCAB)
PAGE = 16               # tokens per KV page
HEAD_DIM = 128
BASE_SEED = 260939334 * 16


@dataclasses.dataclass
class TreeWorkload:
    name: str
    seed: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    # ---- tree (parents before children) -------------------------------------------------------
    node_parent: np.ndarray          # int32 [nodes], -1 for a root
    node_kv_len: np.ndarray          # int32 [nodes]
    node_page_offsets: np.ndarray    # int64 [nodes+1]
    node_pages: np.ndarray           # int32 [sum pages]
    num_pages: int
    # ---- logical candidates, tree order -------------------------------------------------------
    path_leaf_node: np.ndarray       # int32 [N]
    path_q_len: np.ndarray           # int32 [N]  (T: 1 = decode, >1 = verification step)
    path_problem: np.ndarray         # int32 [N]
    dup_of: np.ndarray               # int32 [N]  planted source (-1 if none); NOT a dedup result
    q_offsets: np.ndarray            # int64 [N+1]
    tok_ids: np.ndarray              # int32 [sum leaf lens]  (token ids of each path's own leaf)
    tok_offsets: np.ndarray          # int64 [N+1]
    ctx_key: np.ndarray              # int64 [N]
    slot_in: np.ndarray              # int32 [N]  (= leaf node id)
    # ---- selection ----------------------------------------------------------------------------
    scores: np.ndarray               # float32 [N]
    seg_offsets: np.ndarray          # int32 [P+1]
    top_k: int
    # ---- bulk tensors -------------------------------------------------------------------------
    kv_pool: torch.Tensor            # bf16 [num_pages][2][Hkv][page][D]   (index 0 = K, 1 = V)
    q: torch.Tensor                  # bf16 [total_q][Hq][D]

    @property
    def num_paths(self) -> int:
        return int(self.path_leaf_node.shape[0])

    @property
    def num_nodes(self) -> int:
        return int(self.node_parent.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.q_offsets[-1])

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    # element strides of the pool layout [page][K|V][head][token][dim]
    @property
    def kv_page_stride(self) -> int:
        return 2 * self.num_kv_heads * self.page_size * self.head_dim

    @property
    def kv_head_stride(self) -> int:
        return self.page_size * self.head_dim

    @property
    def kv_token_stride(self) -> int:
        return self.head_dim

    @property
    def v_offset_elems(self) -> int:
        return self.num_kv_heads * self.page_size * self.head_dim

    def chain(self, node: int) -> List[int]:
        """Nodes from the root down to `node`."""
        out = []
        while node >= 0:
            out.append(int(node))
            node = int(self.node_parent[node])
        return out[::-1]

    def path_kv_len(self, p: int) -> int:
        return int(sum(int(self.node_kv_len[n]) for n in self.chain(int(self.path_leaf_node[p]))))


# ------------------------------------------------------------------------------------------------
# bulk fills
# ------------------------------------------------------------------------------------------------
def _randn_bf16(shape: Sequence[int], gen: torch.Generator, device, chunk_elems: int = 1 << 28) -> torch.Tensor:
    """N(0,1) in fp32 rounded to bf16, generated in bounded chunks."""
    n = int(np.prod(shape)) if len(shape) else 1
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    pos = 0
    while pos < n:
        m = min(chunk_elems, n - pos)
        out[pos:pos + m] = torch.randn(m, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
        pos += m
    return out.view(*shape)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns on the host (no value change)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


# ------------------------------------------------------------------------------------------------
# generic builder
# ------------------------------------------------------------------------------------------------
def build_tree_workload(
    name: str,
    seed: int,
    num_q_heads: int,
    num_kv_heads: int,
    level_lens: Sequence[int],
    fanout: Sequence[int],
    n_problems: int,
    leaf_len_range: Tuple[int, int],
    q_len_fn,
    dup_frac: float = 0.0,
    dup_pairs: Optional[Sequence[Tuple[int, int]]] = None,
    top_k: Optional[int] = None,
    device="cpu",
    poison: bool = True,
    tie_heavy_scores: bool = False,
    shuffle_pages: bool = True,
) -> TreeWorkload:
    """Build a tree with `len(level_lens)` shared levels and one leaf level.

    level_lens[l]   KV length of every shared node at level l (level 0 = the problem's prefix)
    fanout[l]       children of each level-l node (the last entry = leaves per lowest shared node)
    q_len_fn(i, n)  query tokens T of sibling i out of n under one lowest shared node's *problem*
    leaf length     U[lo, hi] own suffix (+T for verification paths: the step's own keys are the last T
                    tokens of the leaf)
    dup_frac        that fraction of logical paths are exact copies (token ids, KV, Q) of an earlier
                    sibling with the same parent and the same T
    """
    assert len(level_lens) == len(fanout)
    rng = np.random.Generator(np.random.PCG64(seed))
    D, PG = HEAD_DIM, PAGE

    node_parent: List[int] = []
    node_kv_len: List[int] = []
    path_leaf: List[int] = []
    path_T: List[int] = []
    path_problem: List[int] = []
    path_parent: List[int] = []
    path_sib: List[int] = []            # index among the problem's paths

    paths_per_problem = int(np.prod(fanout))

    def add_node(parent, length):
        node_parent.append(parent)
        node_kv_len.append(length)
        return len(node_parent) - 1

    for pr in range(n_problems):
        counter = [0]

        def rec(level, parent):
            nid = add_node(parent, int(level_lens[level]))
            if level + 1 < len(level_lens):
                for _ in range(fanout[level]):
                    rec(level + 1, nid)
            else:
                for _ in range(fanout[level]):
                    i = counter[0]
                    counter[0] += 1
                    T = int(q_len_fn(i, paths_per_problem, rng))
                    own = int(rng.integers(leaf_len_range[0], leaf_len_range[1] + 1))
                    length = own + (T if T > 1 else 0)
                    leaf = add_node(nid, length)
                    path_leaf.append(leaf)
                    path_T.append(T)
                    path_problem.append(pr)
                    path_parent.append(nid)
                    path_sib.append(i)

        rec(0, -1)

    N = len(path_leaf)
    node_parent_a = np.asarray(node_parent, dtype=np.int32)
    node_kv_len_a = np.asarray(node_kv_len, dtype=np.int32)
    path_leaf_a = np.asarray(path_leaf, dtype=np.int32)
    path_T_a = np.asarray(path_T, dtype=np.int32)
    path_parent_a = np.asarray(path_parent, dtype=np.int32)

    # ---- planted duplicates: copy an earlier, non-duplicate sibling (same parent, same T) ----------
    dup_of = np.full(N, -1, dtype=np.int32)
    if dup_pairs:
        for dst, src in dup_pairs:
            assert src < dst and path_parent_a[src] == path_parent_a[dst]
            dup_of[dst] = src
    elif dup_frac > 0:
        want = int(round(dup_frac * N))
        order = rng.permutation(N)
        # candidates processed in random order; a path may become a duplicate if an earlier sibling of the
        # same parent and T exists that is not itself a duplicate (and is not already a source's copy)
        first_of = {}
        for i in range(N):
            first_of.setdefault((int(path_parent_a[i]), int(path_T_a[i])), []).append(i)
        chosen = 0
        for i in order:
            if chosen >= want:
                break
            sibs = first_of[(int(path_parent_a[i]), int(path_T_a[i]))]
            earlier = [s for s in sibs if s < i and dup_of[s] < 0]
            if not earlier:
                continue
            # a source must stay a non-duplicate: forbid i if something already copies i
            if np.any(dup_of == i):
                continue
            dup_of[i] = earlier[int(rng.integers(0, len(earlier)))]
            chosen += 1
    for i in range(N):
        if dup_of[i] >= 0:
            s = int(dup_of[i])
            node_kv_len_a[path_leaf_a[i]] = node_kv_len_a[path_leaf_a[s]]

    # ---- pages ------------------------------------------------------------------------------------
    n_node_pages = (node_kv_len_a.astype(np.int64) + PG - 1) // PG
    node_page_offsets = np.zeros(len(node_parent) + 1, dtype=np.int64)
    np.cumsum(n_node_pages, out=node_page_offsets[1:])
    num_pages = int(node_page_offsets[-1])
    if shuffle_pages:
        node_pages = rng.permutation(num_pages).astype(np.int32)
    else:
        node_pages = np.arange(num_pages, dtype=np.int32)
    num_pages = max(num_pages, 1)

    # ---- token ids of every path's own leaf ----------------------------------------------------------
    leaf_len = node_kv_len_a[path_leaf_a].astype(np.int64)
    tok_offsets = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(leaf_len, out=tok_offsets[1:])
    tok_ids = rng.integers(0, VOCAB, size=int(tok_offsets[-1]), dtype=np.int64).astype(np.int32)
    for i in range(N):
        if dup_of[i] >= 0:
            s = int(dup_of[i])
            tok_ids[tok_offsets[i]:tok_offsets[i + 1]] = tok_ids[tok_offsets[s]:tok_offsets[s + 1]]
    ctx_key = path_parent_a.astype(np.int64) * 1024 + path_T_a.astype(np.int64)

    q_offsets = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(path_T_a.astype(np.int64), out=q_offsets[1:])

    # ---- scores / segments ------------------------------------------------------------------------------
    if tie_heavy_scores:
        scores = (rng.integers(0, 9, size=N) / 8.0).astype(np.float32)
        scores[rng.random(N) < 0.3] = 1.0
    else:
        scores = rng.random(N, dtype=np.float32)
    seg_offsets = (np.arange(n_problems + 1, dtype=np.int64) * paths_per_problem).astype(np.int32)
    if top_k is None:
        top_k = max(1, paths_per_problem // 4)        # top-k = N / M with beam width M = 4

    # ---- bulk tensors -------------------------------------------------------------------------------------
    gen = torch.Generator(device=device)
    gen.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    kv_pool = _randn_bf16((num_pages, 2, num_kv_heads, PG, D), gen, device)
    total_q = int(q_offsets[-1])
    q = _randn_bf16((max(total_q, 1), num_q_heads, D), gen, device)[:total_q]

    dup_idx = np.nonzero(dup_of >= 0)[0]
    if len(dup_idx):
        dst_pages, src_pages, dst_q, src_q = [], [], [], []
        for i in dup_idx:
            s = int(dup_of[i])
            a, b = node_page_offsets[path_leaf_a[i]], node_page_offsets[path_leaf_a[i] + 1]
            c, d = node_page_offsets[path_leaf_a[s]], node_page_offsets[path_leaf_a[s] + 1]
            assert b - a == d - c
            dst_pages.append(node_pages[a:b]); src_pages.append(node_pages[c:d])
            dst_q.append(np.arange(q_offsets[i], q_offsets[i + 1])); src_q.append(np.arange(q_offsets[s], q_offsets[s + 1]))
        dp = torch.from_numpy(np.concatenate(dst_pages).astype(np.int64)).to(device)
        sp = torch.from_numpy(np.concatenate(src_pages).astype(np.int64)).to(device)
        if dp.numel():
            kv_pool[dp] = kv_pool[sp]
        dq = torch.from_numpy(np.concatenate(dst_q).astype(np.int64)).to(device)
        sq = torch.from_numpy(np.concatenate(src_q).astype(np.int64)).to(device)
        if dq.numel():
            q[dq] = q[sq]

    if poison:
        # slots past a node's length in its last page are undefined: fill with NaN so that any read of them
        # into a result shows up
        rem = node_kv_len_a.astype(np.int64) % PG
        partial = np.nonzero((rem != 0))[0]
        if len(partial):
            last_page = node_pages[node_page_offsets[partial + 1] - 1].astype(np.int64)
            rows = np.arange(PG)[None, :]
            mask = rows >= rem[partial][:, None]
            pi, ri = np.nonzero(mask)
            pidx = torch.from_numpy(last_page[pi]).to(device)
            ridx = torch.from_numpy(ri.astype(np.int64)).to(device)
            kv_pool[pidx, :, :, ridx, :] = float("nan")

    return TreeWorkload(
        name=name, seed=seed, num_q_heads=num_q_heads, num_kv_heads=num_kv_heads, head_dim=D, page_size=PG,
        node_parent=node_parent_a, node_kv_len=node_kv_len_a, node_page_offsets=node_page_offsets,
        node_pages=node_pages, num_pages=num_pages,
        path_leaf_node=path_leaf_a, path_q_len=path_T_a, path_problem=np.asarray(path_problem, dtype=np.int32),
        dup_of=dup_of, q_offsets=q_offsets, tok_ids=tok_ids, tok_offsets=tok_offsets, ctx_key=ctx_key,
        slot_in=path_leaf_a.copy(), scores=scores, seg_offsets=seg_offsets, top_k=int(top_k),
        kv_pool=kv_pool, q=q,
    )


# ------------------------------------------------------------------------------------------------
# the five benchmark configurations
# ------------------------------------------------------------------------------------------------
def _decode(i, n, rng):
    return 1


def make_config(idx: int, device="cpu", scale: float = 1.0, poison: bool = True, replica: int = 0) -> TreeWorkload:
    """Config 1..5 of the benchmark list.  `scale` < 1 shrinks the number of problems (tests only); `replica`
    selects a different seed for the same shapes (one replica per GPU in a multi-GPU run)."""
    seed = BASE_SEED + idx + 1000 * replica
    if idx == 1:
        # 1 problem, 8 paths sharing a 256-token prefix, suffix U[0,64], decode; 12/2 heads; 2 of 8 identical
        return build_tree_workload("c1_tiny", seed, 12, 2, [256], [8], 1, (0, 64), _decode,
                                   dup_pairs=[(7, 3)], top_k=2, device=device, poison=poison)
    if idx == 2:
        P = max(1, int(round(16 * scale)))
        return build_tree_workload("c2_expansion_decode", seed, 12, 2, [512], [64], P, (32, 512), _decode,
                                   dup_frac=0.10, top_k=16, device=device, poison=poison)
    if idx == 3:
        P = max(1, int(round(8 * scale)))
        return build_tree_workload("c3_verification", seed, 28, 4, [1024], [32], P, (64, 512),
                                   lambda i, n, rng: int(rng.integers(16, 129)),
                                   dup_frac=0.0, top_k=8, device=device, poison=poison)
    if idx == 4:
        P = max(1, int(round(4 * scale)))
        return build_tree_workload("c4_two_level", seed, 32, 8, [2048, 256], [16, 16], P, (64, 256), _decode,
                                   dup_frac=0.30, top_k=64, device=device, poison=poison)
    if idx == 5:
        P = max(1, int(round(64 * scale)))
        return build_tree_workload("c5_large_mixed", seed, 32, 8, [4096], [256], P, (128, 1024),
                                   lambda i, n, rng: 1 if i < n // 2 else 64,
                                   dup_frac=0.20, top_k=64, device=device, poison=poison)
    raise ValueError(f"unknown config {idx}")


# ------------------------------------------------------------------------------------------------
# selecting / compacting paths (plain gathers; used to hand the unique paths to the attention call and to
# cut a sample out of a large workload for the CPU oracle)
# ------------------------------------------------------------------------------------------------
def select_paths(w: TreeWorkload, keep: np.ndarray) -> Dict[str, np.ndarray]:
    """Per-path descriptor arrays restricted to `keep` (ascending logical indices), plus the gather index
    of their query rows."""
    keep = np.asarray(keep, dtype=np.int64)
    T = w.path_q_len[keep].astype(np.int64)
    q_off = np.zeros(len(keep) + 1, dtype=np.int64)
    np.cumsum(T, out=q_off[1:])
    rows = np.concatenate([np.arange(w.q_offsets[i], w.q_offsets[i + 1]) for i in keep]) if len(keep) else \
        np.zeros(0, dtype=np.int64)
    return dict(path_leaf_node=w.path_leaf_node[keep].copy(), path_q_len=w.path_q_len[keep].copy(),
                q_offsets=q_off, q_rows=rows.astype(np.int64))


def extract_subworkload(w: TreeWorkload, keep: np.ndarray) -> TreeWorkload:
    """A self-contained host copy of the paths in `keep`: only the nodes on their chains and only the pages
    of those nodes (page ids renumbered densely).  Used to feed a sample of a large device-resident workload
    to the CPU oracle."""
    keep = np.asarray(sorted(int(i) for i in keep), dtype=np.int64)
    used_nodes = sorted({n for p in keep for n in w.chain(int(w.path_leaf_node[p]))})
    remap = {n: j for j, n in enumerate(used_nodes)}
    un = np.asarray(used_nodes, dtype=np.int64)
    node_parent = np.asarray([remap[int(w.node_parent[n])] if w.node_parent[n] >= 0 else -1 for n in used_nodes],
                             dtype=np.int32)
    node_kv_len = w.node_kv_len[un].copy()
    cnt = (w.node_page_offsets[un + 1] - w.node_page_offsets[un]).astype(np.int64)
    node_page_offsets = np.zeros(len(un) + 1, dtype=np.int64)
    np.cumsum(cnt, out=node_page_offsets[1:])
    old_pages = np.concatenate([w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]] for n in used_nodes]) \
        if len(used_nodes) else np.zeros(0, dtype=np.int32)
    new_pages = np.arange(len(old_pages), dtype=np.int32)
    sel = select_paths(w, keep)
    idx = torch.from_numpy(old_pages.astype(np.int64)).to(w.kv_pool.device)
    kv_pool = w.kv_pool[idx].cpu() if len(old_pages) else w.kv_pool[:1].cpu()
    qidx = torch.from_numpy(sel["q_rows"]).to(w.q.device)
    q = w.q[qidx].cpu()
    tok_off = np.zeros(len(keep) + 1, dtype=np.int64)
    np.cumsum(w.tok_offsets[keep + 1] - w.tok_offsets[keep], out=tok_off[1:])
    tok = np.concatenate([w.tok_ids[w.tok_offsets[i]:w.tok_offsets[i + 1]] for i in keep]) if len(keep) else \
        np.zeros(0, dtype=np.int32)
    leaf = np.asarray([remap[int(n)] for n in sel["path_leaf_node"]], dtype=np.int32)
    return TreeWorkload(
        name=w.name + "_sample", seed=w.seed, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads,
        head_dim=w.head_dim, page_size=w.page_size, node_parent=node_parent, node_kv_len=node_kv_len,
        node_page_offsets=node_page_offsets, node_pages=new_pages, num_pages=max(1, len(old_pages)),
        path_leaf_node=leaf, path_q_len=sel["path_q_len"], path_problem=w.path_problem[keep].copy(),
        dup_of=np.full(len(keep), -1, dtype=np.int32), q_offsets=sel["q_offsets"], tok_ids=tok.astype(np.int32),
        tok_offsets=tok_off, ctx_key=w.ctx_key[keep].copy(), slot_in=leaf.copy(), scores=w.scores[keep].copy(),
        seg_offsets=np.asarray([0, len(keep)], dtype=np.int32), top_k=w.top_k, kv_pool=kv_pool, q=q)
