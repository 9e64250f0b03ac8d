"""Pins for the CPU oracle: it is checked against things other than itself - the paper's worked examples
(tests/golden), brute force written a second way, closed forms, invariants and a library routine."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# =========================================================================================================
# helpers (written independently of the oracle)
# =========================================================================================================
def csr(seqs):
    off = np.zeros(len(seqs) + 1, np.int64)
    for i, s in enumerate(seqs):
        off[i + 1] = off[i] + len(s)
    ids = np.asarray([t for s in seqs for t in s], np.int32)
    return ids, off


def brute_dedup(seqs, ctx):
    """O(N^2) pairwise comparison."""
    n = len(seqs)
    canon = list(range(n))
    for i in range(n):
        for j in range(i):
            if ctx[j] == ctx[i] and list(seqs[j]) == list(seqs[i]):
                canon[i] = j
                break
    uniq = [i for i in range(n) if canon[i] == i]
    rank = {u: r for r, u in enumerate(uniq)}
    p2u = [rank[canon[i]] for i in range(n)]
    mult = [sum(1 for i in range(n) if canon[i] == u) for u in uniq]
    return canon, p2u, uniq, mult


def random_seqs(rng, n, alphabet=3, max_len=4, n_ctx=2):
    seqs = [list(rng.integers(0, alphabet, size=int(rng.integers(0, max_len + 1)))) for _ in range(n)]
    ctx = [int(rng.integers(0, n_ctx)) for _ in range(n)]
    return seqs, ctx


def gather_path_kv(w, p):
    """(K, V) of path p as float64 [L][Hkv][D], by walking the chain - numpy indexing, not the oracle's loop."""
    pool = w.kv_pool.to(torch.float64).numpy()
    ks, vs = [], []
    for n in w.chain(int(w.path_leaf_node[p])):
        L = int(w.node_kv_len[n])
        pages = w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]]
        if L == 0:
            continue
        blk = pool[pages]                                  # [np][2][Hkv][16][D]
        k = np.transpose(blk[:, 0], (0, 2, 1, 3)).reshape(-1, w.num_kv_heads, w.head_dim)[:L]
        v = np.transpose(blk[:, 1], (0, 2, 1, 3)).reshape(-1, w.num_kv_heads, w.head_dim)[:L]
        ks.append(k)
        vs.append(v)
    if not ks:
        z = np.zeros((0, w.num_kv_heads, w.head_dim))
        return z, z
    return np.concatenate(ks), np.concatenate(vs)


def levelwise_attention(w, scale):
    """Second, independent evaluation: per tree level a partial (o, lse); partials merged with the
    log-sum-exp identity.  Mirrors how a level-split kernel works, not how the oracle works."""
    q = w.q.to(torch.float64).numpy()
    pool = w.kv_pool.to(torch.float64).numpy()
    G = w.group
    out = np.zeros((w.total_q, w.num_q_heads, w.head_dim))
    lse = np.full((w.total_q, w.num_q_heads), -np.inf)
    for p in range(w.num_paths):
        chain = w.chain(int(w.path_leaf_node[p]))
        T = int(w.path_q_len[p])
        L = sum(int(w.node_kv_len[n]) for n in chain)
        for t in range(T):
            row = int(w.q_offsets[p]) + t
            visible = L - T + t + 1
            for h in range(w.num_q_heads):
                g = h // G
                parts = []
                start = 0
                for n in chain:
                    ln = int(w.node_kv_len[n])
                    cnt = min(ln, max(0, visible - start))
                    if cnt > 0:
                        pages = w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]]
                        k = pool[pages, 0, g].reshape(-1, w.head_dim)[:cnt]
                        v = pool[pages, 1, g].reshape(-1, w.head_dim)[:cnt]
                        s = scale * (k @ q[row, h])
                        m = s.max()
                        e = np.exp(s - m)
                        parts.append((e @ v / e.sum(), m + math.log(e.sum())))
                    start += ln
                if parts:
                    ls = np.array([pl for _, pl in parts])
                    tot = ls.max() + math.log(np.exp(ls - ls.max()).sum())
                    out[row, h] = sum(np.exp(pl - tot) * po for po, pl in parts)
                    lse[row, h] = tot
    return out, lse


def small_tree(seed, Hq=4, Hkv=2, levels=(32,), fanout=(3,), problems=2, leaf=(0, 40), qfn=None, dup=0.0,
               poison=True):
    if qfn is None:
        qfn = lambda i, n, rng: 1
    return synth.build_tree_workload("t", seed, Hq, Hkv, list(levels), list(fanout), problems, leaf, qfn,
                                     dup_frac=dup, poison=poison)


SCALE = 1.0 / math.sqrt(128.0)


# =========================================================================================================
# dedup
# =========================================================================================================
def test_dedup_paper_worked_example():
    with open(os.path.join(GOLDEN, "dedup_on_demand_branching.txt")) as f:
        lines = [l.strip() for l in f if l.strip() and not l.startswith("#")]
    assert lines
    for line in lines:
        left, right = line.split("|")
        samples = [int(x) for x in left.split(":")[1].split()]
        potentials = [int(x) for x in right.split(":")[1].split()]
        # each child sequence = (shared parent context, sampled token)
        ids, off = csr([[s] for s in samples])
        r = oracle.dedup(ids, off, ctx_key=np.zeros(len(samples), np.int64))
        assert r["num_unique"] == len(potentials)
        assert list(r["multiplicity"]) == potentials
        assert sum(potentials) == len(samples)


@pytest.mark.parametrize("seed", range(6))
def test_dedup_bruteforce(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 64))
    seqs, ctx = random_seqs(rng, n)
    ids, off = csr(seqs)
    slot = rng.integers(0, 1000, size=n).astype(np.int32)
    r = oracle.dedup(ids, off, ctx_key=np.asarray(ctx, np.int64), slot_in=slot)
    canon, p2u, uniq, mult = brute_dedup(seqs, ctx)
    assert list(r["canon"]) == canon
    assert list(r["path_to_unique"]) == p2u
    assert list(r["unique_paths"]) == uniq
    assert list(r["multiplicity"]) == mult
    assert list(r["slot_out"]) == [int(slot[c]) for c in canon]
    assert r["num_unique"] == len({(c, tuple(s)) for c, s in zip(ctx, seqs)})
    assert int(r["multiplicity"].sum()) == n


def test_dedup_ctx_key_separates_and_null_ctx():
    ids, off = csr([[1, 2], [1, 2], [1, 2]])
    r = oracle.dedup(ids, off, ctx_key=np.asarray([0, 1, 0], np.int64))
    assert list(r["canon"]) == [0, 1, 0]
    r = oracle.dedup(ids, off)
    assert list(r["canon"]) == [0, 0, 0]
    # prefix of a sequence is not the sequence; empty sequences are duplicates of each other
    ids, off = csr([[1, 2], [1], [], [1, 2, 3], []])
    r = oracle.dedup(ids, off)
    assert list(r["canon"]) == [0, 1, 2, 3, 2]


@pytest.mark.parametrize("seed", range(4))
def test_dedup_idempotent(seed):
    rng = np.random.default_rng(100 + seed)
    seqs, ctx = random_seqs(rng, 50)
    ids, off = csr(seqs)
    r = oracle.dedup(ids, off, ctx_key=np.asarray(ctx, np.int64))
    useqs = [seqs[u] for u in r["unique_paths"]]
    uctx = [ctx[u] for u in r["unique_paths"]]
    ids2, off2 = csr(useqs)
    r2 = oracle.dedup(ids2, off2, ctx_key=np.asarray(uctx, np.int64))
    U = r["num_unique"]
    assert r2["num_unique"] == U
    assert list(r2["canon"]) == list(range(U))
    assert list(r2["multiplicity"]) == [1] * U


@pytest.mark.parametrize("seed", range(4))
def test_dedup_permutation_invariance(seed):
    rng = np.random.default_rng(200 + seed)
    n = 40
    seqs, ctx = random_seqs(rng, n)
    ids, off = csr(seqs)
    r = oracle.dedup(ids, off, ctx_key=np.asarray(ctx, np.int64))
    perm = rng.permutation(n)                 # new position j holds old path perm[j]
    inv = np.argsort(perm)
    ids2, off2 = csr([seqs[i] for i in perm])
    r2 = oracle.dedup(ids2, off2, ctx_key=np.asarray([ctx[i] for i in perm], np.int64))
    assert r2["num_unique"] == r["num_unique"]
    # classes map through the permutation and the canonical is the class minimum in the new order
    classes = {}
    for i in range(n):
        classes.setdefault(int(r["canon"][i]), []).append(int(inv[i]))
    for members in classes.values():
        for j in members:
            assert int(r2["canon"][j]) == min(members)


def test_dedup_config1_generator():
    w = synth.make_config(1)
    r = oracle.dedup(w.tok_ids, w.tok_offsets, ctx_key=w.ctx_key, slot_in=w.slot_in)
    assert int(r["canon"][7]) == 3            # the planted pair
    keys = {(int(c), tuple(w.tok_ids[w.tok_offsets[i]:w.tok_offsets[i + 1]])) for i, c in enumerate(w.ctx_key)}
    assert r["num_unique"] == len(keys)
    assert int(r["slot_out"][7]) == int(w.slot_in[3])


# =========================================================================================================
# attention
# =========================================================================================================
@pytest.mark.parametrize("cfg", [
    dict(seed=1),
    dict(seed=2, Hq=6, Hkv=2, levels=(16, 32), fanout=(2, 2), problems=1, leaf=(0, 20)),
    dict(seed=3, Hq=4, Hkv=1, levels=(48,), fanout=(2,), problems=2, leaf=(5, 30),
         qfn=lambda i, n, rng: int(rng.integers(2, 9))),
    dict(seed=4, Hq=2, Hkv=2, levels=(16,), fanout=(3,), problems=1, leaf=(0, 3),
         qfn=lambda i, n, rng: 1 + (i % 2) * 4),
])
def test_attention_vs_levelwise_bruteforce(cfg):
    w = small_tree(**cfg)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE, n_threads=2)
    ref_out, ref_lse = levelwise_attention(w, SCALE)
    assert np.isfinite(out).all()
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=0, atol=1e-12)


def test_attention_split_merge_identity_arbitrary_splits():
    """Softmax over a key set equals the log-sum-exp merge of softmaxes over any partition of it."""
    rng = np.random.default_rng(7)
    w = small_tree(11, Hq=2, Hkv=1, levels=(64,), fanout=(1,), problems=1, leaf=(33, 33), poison=False)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE, n_threads=1)
    K, V = gather_path_kv(w, 0)
    q = w.q.to(torch.float64).numpy()
    L = K.shape[0]
    for trial in range(5):
        labels = rng.integers(0, 4, size=L)
        for h in range(2):
            parts = []
            for lab in range(4):
                sel = labels == lab
                if not sel.any():
                    continue
                s = SCALE * (K[sel, 0] @ q[0, h])
                m = s.max()
                e = np.exp(s - m)
                parts.append((e @ V[sel, 0] / e.sum(), m + math.log(e.sum())))
            ls = np.array([p[1] for p in parts])
            tot = ls.max() + math.log(np.exp(ls - ls.max()).sum())
            merged = sum(np.exp(p[1] - tot) * p[0] for p in parts)
            np.testing.assert_allclose(merged, out[0, h], atol=1e-12)
            assert abs(tot - lse[0, h]) < 1e-12


def test_attention_tree_restructure_invariance():
    """Cutting a node in two at a page boundary (same tokens, same order) changes nothing."""
    w = small_tree(21, Hq=4, Hkv=2, levels=(64,), fanout=(2,), problems=1, leaf=(1, 30),
                   qfn=lambda i, n, rng: 3, poison=False)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    # new tree: root split into 2 nodes of 32 tokens
    w2 = small_tree(21, Hq=4, Hkv=2, levels=(64,), fanout=(2,), problems=1, leaf=(1, 30),
                    qfn=lambda i, n, rng: 3, poison=False)
    root_pages = w.node_pages[w.node_page_offsets[0]:w.node_page_offsets[1]]
    node_parent = np.asarray([-1, 0] + [p + 1 if p >= 0 else -1 for p in w.node_parent[1:]], np.int32)
    node_parent[2:] = np.where(w.node_parent[1:] == 0, 1, w.node_parent[1:] + 1)
    node_kv_len = np.asarray([32, 32] + list(w.node_kv_len[1:]), np.int32)
    node_pages = np.concatenate([root_pages[:2], root_pages[2:], w.node_pages[w.node_page_offsets[1]:]]).astype(np.int32)
    offs = np.zeros(len(node_kv_len) + 1, np.int64)
    np.cumsum((node_kv_len + 15) // 16, out=offs[1:])
    w2.node_parent, w2.node_kv_len, w2.node_pages, w2.node_page_offsets = node_parent, node_kv_len, node_pages, offs
    w2.path_leaf_node = w.path_leaf_node + 1
    out2, lse2 = oracle.tree_attention_workload(w2, sm_scale=SCALE)
    np.testing.assert_allclose(out2, out, atol=1e-13)
    np.testing.assert_allclose(lse2, lse, atol=1e-13)


def test_attention_rows_sum_to_one():
    w = small_tree(31, Hq=6, Hkv=2, levels=(32,), fanout=(4,), problems=2, leaf=(0, 50),
                   qfn=lambda i, n, rng: 1 + 3 * (i % 2), poison=False)
    w.kv_pool[:, 1] = 1.0
    out, _ = oracle.tree_attention_workload(w, sm_scale=SCALE)
    np.testing.assert_allclose(out, 1.0, atol=1e-12)


@pytest.mark.parametrize("T", [1, 5, 16])
def test_attention_vs_torch_sdpa_single_path(T):
    """One path, one node: the library routine with an explicit bottom-right causal mask and repeated kv heads."""
    L = 40
    w = synth.build_tree_workload("s", 41 + T, 6, 2, [0], [1], 1, (L - (T if T > 1 else 0),) * 2,
                                  lambda i, n, rng: T, poison=False)
    assert w.path_kv_len(0) == L
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    K, V = gather_path_kv(w, 0)
    q = w.q.to(torch.float64)                                    # [T][Hq][D]
    kt = torch.from_numpy(K).repeat_interleave(3, dim=1)         # [L][Hq][D]
    vt = torch.from_numpy(V).repeat_interleave(3, dim=1)
    mask = torch.zeros(T, L, dtype=torch.bool)
    for t in range(T):
        mask[t, :L - T + t + 1] = True
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.permute(1, 0, 2)[None], kt.permute(1, 0, 2)[None], vt.permute(1, 0, 2)[None], attn_mask=mask, scale=SCALE)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    s = SCALE * torch.einsum("thd,lhd->htl", q, kt).masked_fill(~mask[None], float("-inf"))
    np.testing.assert_allclose(lse, torch.logsumexp(s, dim=-1).T.numpy(), atol=1e-12)


@pytest.mark.parametrize("levels,fanout,T", [((32,), (3,), 1), ((16, 32), (2, 2), 1), ((48,), (2,), 7)])
def test_attention_closed_forms(levels, fanout, T):
    """Q == 0  =>  lse = ln(#visible keys), out = mean of visible V rows.  With V[j, :] = j (j = position in
    the path) the mean is (L-T+t)/2: any off-by-one in mask, page order or node length changes it.
    Values are kept below 256 so that bf16 holds them exactly."""
    w = small_tree(51, Hq=4, Hkv=2, levels=levels, fanout=fanout, problems=1, leaf=(0, 60),
                   qfn=lambda i, n, rng: T, poison=True)
    w.q.zero_()
    pool = w.kv_pool
    for p in range(w.num_paths):
        pos = 0
        for n in w.chain(int(w.path_leaf_node[p])):
            pages = w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]]
            for j in range(int(w.node_kv_len[n])):
                pool[int(pages[j // 16]), 1, :, j % 16, :] = float(pos)
                pos += 1
        assert pos < 256
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    for p in range(w.num_paths):
        L = w.path_kv_len(p)
        for t in range(T):
            row = int(w.q_offsets[p]) + t
            vis = L - T + t + 1
            if vis <= 0:
                assert np.all(out[row] == 0) and np.all(np.isneginf(lse[row]))
                continue
            np.testing.assert_allclose(lse[row], math.log(vis), atol=1e-13)
            np.testing.assert_allclose(out[row], (vis - 1) / 2.0, atol=1e-11)


def test_attention_constant_k_same_closed_form():
    w = small_tree(52, Hq=4, Hkv=2, levels=(32,), fanout=(2,), problems=1, leaf=(1, 20), poison=False)
    w.kv_pool[:, 0] = 0.5
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    q = w.q.to(torch.float64).numpy()
    for p in range(w.num_paths):
        L = w.path_kv_len(p)
        K, V = gather_path_kv(w, p)
        row = int(w.q_offsets[p])
        for h in range(4):
            s = SCALE * 0.5 * q[row, h].sum()
            assert abs(lse[row, h] - (s + math.log(L))) < 1e-12
            np.testing.assert_allclose(out[row, h], V[:, h // 2].mean(axis=0), atol=1e-12)


def test_attention_empty_path_defined():
    w = synth.build_tree_workload("e", 61, 2, 1, [0], [2], 1, (0, 0), lambda i, n, rng: 1)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    assert np.all(out == 0) and np.all(np.isneginf(lse))


def test_attention_page_permutation_bit_identical_and_poison_never_read():
    w = small_tree(71, Hq=4, Hkv=2, levels=(32,), fanout=(3,), problems=2, leaf=(1, 40),
                   qfn=lambda i, n, rng: 1 + 2 * (i % 2), poison=True)
    assert torch.isnan(w.kv_pool.float()).any()          # poison present in unused slots
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    rng = np.random.default_rng(0)
    perm = rng.permutation(w.num_pages)                   # new id of old page i is perm[i]
    new_pool = torch.empty_like(w.kv_pool)
    new_pool[torch.from_numpy(perm)] = w.kv_pool
    w.kv_pool = new_pool
    w.node_pages = perm[w.node_pages].astype(np.int32)
    out2, lse2 = oracle.tree_attention_workload(w, sm_scale=SCALE)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_attention_duplicate_paths_equal_outputs():
    w = synth.make_config(1)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    assert np.array_equal(out[7], out[3]) and np.array_equal(lse[7], lse[3])
    sub, sub_lse = oracle.tree_attention_workload(w, paths=[3, 5], sm_scale=SCALE)
    assert np.array_equal(sub[0], out[3]) and np.array_equal(sub[1], out[5])


def test_attention_strided_pool_layout_equivalence():
    """The pool is described by strides: a token-major [page][token][head][dim] copy gives the same result."""
    w = small_tree(81, Hq=4, Hkv=2, levels=(32,), fanout=(2,), problems=1, leaf=(1, 20), poison=False)
    out, lse = oracle.tree_attention_workload(w, sm_scale=SCALE)
    k = w.kv_pool[:, 0].permute(0, 2, 1, 3).contiguous()   # [page][token][head][dim]
    v = w.kv_pool[:, 1].permute(0, 2, 1, 3).contiguous()
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    out2, lse2 = oracle.tree_attention(4, 2, 128, 16, SCALE, bits(k), bits(v), 16 * 2 * 128, 128, 2 * 128,
                                       w.node_parent, w.node_kv_len, w.node_page_offsets, w.node_pages,
                                       w.path_leaf_node, w.path_q_len, w.q_offsets, bits(w.q))
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


# =========================================================================================================
# top-k
# =========================================================================================================
def brute_topk(scores, seg, k):
    surv = np.full((len(seg) - 1, k), -1, np.int32)
    keep = np.zeros(len(scores), np.uint8)
    for s in range(len(seg) - 1):
        idx = list(range(seg[s], seg[s + 1]))
        key = []
        for i in idx:
            x = float(scores[i])
            key.append((1 if math.isnan(x) else 0, 0.0 if math.isnan(x) else -(x + 0.0), i))
        order = [t[2] for t in sorted(key)]
        for j, i in enumerate(order[:k]):
            surv[s, j] = i
            keep[i] = 1
    return surv, keep


def test_topk_beam_bookkeeping_golden():
    with open(os.path.join(GOLDEN, "topk_beam_bookkeeping.txt")) as f:
        rows = [tuple(int(x) for x in l.split()) for l in f if l.strip() and not l.startswith("#")]
    assert (4, 4, 1) in rows
    rng = np.random.default_rng(5)
    for N, M, k in rows:
        assert k == N // M
        sc = rng.random(N).astype(np.float32)
        surv, keep = oracle.topk(sc, [0, N], k)
        assert int(keep.sum()) == k
        assert set(surv[0]) == set(np.argsort(-sc, kind="stable")[:k])


@pytest.mark.parametrize("seed", range(5))
def test_topk_bruteforce_and_invariants(seed):
    rng = np.random.default_rng(300 + seed)
    sizes = rng.integers(0, 40, size=6)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    n = int(seg[-1])
    sc = (rng.integers(0, 9, size=n) / 8.0).astype(np.float32)       # tie-heavy 1/8 grid
    sc[rng.random(n) < 0.3] = 1.0                                    # large mass at the perfect score
    k = int(rng.integers(1, 12))
    surv, keep = oracle.topk(sc, seg, k)
    bs, bk = brute_topk(sc, seg, k)
    assert np.array_equal(surv, bs) and np.array_equal(keep, bk)
    for s in range(len(sizes)):
        lo, hi = seg[s], seg[s + 1]
        kept = [i for i in range(lo, hi) if keep[i]]
        dropped = [i for i in range(lo, hi) if not keep[i]]
        assert len(kept) == min(k, hi - lo)
        if kept and dropped:
            assert min(sc[kept]) >= max(sc[dropped])
            # ties at the boundary go to the lower index
            b = min(sc[kept])
            assert all(i > max(j for j in kept if sc[j] == b) for i in dropped if sc[i] == b)


def test_topk_special_values():
    sc = np.asarray([0.0, -0.0, np.nan, 0.5, np.nan, -1.0, np.inf, -np.inf], np.float32)
    surv, keep = oracle.topk(sc, [0, 8], 8)
    assert list(surv[0]) == [6, 3, 0, 1, 5, 7, 2, 4]
    surv, keep = oracle.topk(sc, [0, 8], 3)
    assert list(surv[0]) == [6, 3, 0] and list(keep) == [1, 0, 0, 1, 0, 0, 1, 0]
    surv, keep = oracle.topk(sc[:2], [0, 2], 4)
    assert list(surv[0]) == [0, 1, -1, -1]


# =========================================================================================================
# generators: structure checks (so that the pins above run on the intended shapes)
# =========================================================================================================
def test_generator_shapes_config2_small():
    w = synth.make_config(2, scale=1 / 16)
    assert w.num_paths == 64 and w.num_q_heads == 12 and w.num_kv_heads == 2
    assert int(w.node_kv_len[0]) == 512
    n_dup = int((w.dup_of >= 0).sum())
    assert n_dup == round(0.10 * 64)
    for i in np.nonzero(w.dup_of >= 0)[0]:
        s = int(w.dup_of[i])
        a = w.tok_ids[w.tok_offsets[i]:w.tok_offsets[i + 1]]
        b = w.tok_ids[w.tok_offsets[s]:w.tok_offsets[s + 1]]
        assert np.array_equal(a, b) and w.ctx_key[i] == w.ctx_key[s]
        assert torch.equal(w.q[int(w.q_offsets[i])].view(torch.int16), w.q[int(w.q_offsets[s])].view(torch.int16))
    # DFS order: the paths below every node are contiguous
    for n in range(w.num_nodes):
        below = [p for p in range(w.num_paths) if n in w.chain(int(w.path_leaf_node[p]))]
        if below:
            assert below == list(range(below[0], below[-1] + 1))


# =========================================================================================================
# early pruning with partially verified candidates
# =========================================================================================================
def brute_early_prune(scores, verified, seg, k):
    n = len(scores)
    pruned = np.zeros(n, np.uint8)
    sel = np.full((len(seg) - 1, k), -1, np.int32)
    fin = np.zeros(len(seg) - 1, np.uint8)
    for s in range(len(seg) - 1):
        idx = list(range(seg[s], seg[s + 1]))
        ver = [i for i in idx if verified[i]]
        perfect = [i for i in ver if scores[i] >= 1.0]
        if len(perfect) >= k:
            chosen = perfect[:k]
            for i in idx:
                pruned[i] = 0 if i in chosen else 1
            sel[s, :k] = chosen
            fin[s] = 1
            continue
        order = sorted(ver, key=lambda i: (1 if math.isnan(scores[i]) else 0,
                                           0.0 if math.isnan(scores[i]) else -(float(scores[i]) + 0.0), i))
        if len(ver) > k:
            for i in order[k:]:
                pruned[i] = 1
        if len(ver) == len(idx):
            fin[s] = 1
            sel[s, :min(k, len(order))] = order[:k]
    return pruned, sel, fin


def test_early_prune_paper_worked_example():
    """The figure's walk-through: k = 1; B verified -> continues; D verified lower -> pruned; C perfect -> all others
    pruned and C selected."""
    lines = [l.strip() for l in open(os.path.join(GOLDEN, "early_pruning_example.txt")) if l.strip() and not l.startswith("#")]
    k = int(lines[0].split()[1])
    names = lines[1].split()[1:]
    scores = np.zeros(len(names), np.float32)
    verified = np.zeros(len(names), np.uint8)
    seg = np.asarray([0, len(names)], np.int32)
    cumulative_pruned = set()
    for line in lines[2:]:
        ev, pr, se = [x.strip() for x in line.split("|")]
        _, who, val = ev.split()
        scores[names.index(who)] = float(val)
        verified[names.index(who)] = 1
        pruned, sel, fin = oracle.early_prune(scores, verified, seg, k)
        cumulative_pruned |= {names[i] for i in range(len(names)) if pruned[i]}
        want_pruned = set() if pr.split(":")[1].strip() == "-" else set(pr.split(":")[1].split())
        assert cumulative_pruned == want_pruned, line
        want_sel = se.split(":")[1].strip()
        if want_sel == "-":
            assert fin[0] == 0 and list(sel[0]) == [-1] * k
        else:
            assert fin[0] == 1 and [names[i] for i in sel[0]] == want_sel.split()


@pytest.mark.parametrize("seed", range(6))
def test_early_prune_bruteforce_and_topk_consistency(seed):
    rng = np.random.default_rng(400 + seed)
    sizes = rng.integers(0, 30, size=7)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    n = int(seg[-1])
    sc = (rng.integers(0, 9, size=n) / 8.0).astype(np.float32)
    sc[rng.random(n) < 0.25] = 1.0
    k = int(rng.integers(1, 6))
    for frac in (0.0, 0.3, 0.7, 1.0):
        ver = (rng.random(n) < frac).astype(np.uint8) if frac < 1.0 else np.ones(n, np.uint8)
        pruned, sel, fin = oracle.early_prune(sc, ver, seg, k)
        bp, bs, bf = brute_early_prune(sc, ver, seg, k)
        assert np.array_equal(pruned, bp) and np.array_equal(sel, bs) and np.array_equal(fin, bf)
        # an unverified candidate is only ever pruned by rule 2 (segment final through perfect scores)
        for s in range(len(sizes)):
            for i in range(seg[s], seg[s + 1]):
                if pruned[i] and not ver[i]:
                    assert fin[s] == 1
    # everything verified and fewer than k perfect scores in a segment => same survivors as the plain top-k
    ver = np.ones(n, np.uint8)
    sc2 = np.minimum(sc, np.float32(0.875))
    pruned, sel, fin = oracle.early_prune(sc2, ver, seg, k)
    surv, keep = oracle.topk(sc2, seg, k)
    assert np.array_equal(1 - pruned, keep) and np.array_equal(sel, surv) and fin.all()


# =========================================================================================================
# on-demand branching: sampling
# =========================================================================================================
def test_branch_sample_paper_worked_example():
    kv = {}
    for l in open(os.path.join(GOLDEN, "branch_sampling_example.txt")):
        if l.strip() and not l.startswith("#"):
            k, *v = l.split()
            kv[k] = v
    probs = np.asarray([float(x) for x in kv["probs"]])
    with np.errstate(divide="ignore"):
        logits = np.log(probs).astype(np.float32)[None, :]            # -inf where the probability is zero
    u = np.asarray([float(x) for x in kv["uniforms"]], np.float32)
    tokens, seq, _ = oracle.branch_sample(logits, [0, len(u)], u, float(kv["temperature"][0]))
    assert list(tokens) == [int(x) for x in kv["tokens"]] and set(seq) == {0}
    # grouping of the draws = dedup of (sequence, token) pairs; cardinalities = the children's potential sizes
    r = oracle.dedup(tokens, np.arange(len(u) + 1), ctx_key=seq)
    assert list(r["multiplicity"]) == [int(x) for x in kv["potentials"]]


def test_branch_sample_closed_forms():
    rng = np.random.default_rng(3)
    V = 1000
    u = rng.random(500).astype(np.float32)
    # uniform logits: token = floor(u * V)
    tokens, _, margin = oracle.branch_sample(np.zeros((1, V), np.float32), [0, 500], u, 0.7)
    safe = margin > 1e-9
    assert np.array_equal(tokens[safe], np.floor(u.astype(np.float64) * V).astype(np.int32)[safe])
    # one token carries everything: always that token, whatever the temperature
    lg = np.full((1, V), -np.inf, np.float32)
    lg[0, 417] = 3.0
    assert set(oracle.branch_sample(lg, [0, 500], u, 2.0)[0]) == {417}
    # scaling logits and temperature together changes nothing; sorted uniforms give non-decreasing tokens
    lg = rng.normal(size=(1, V)).astype(np.float32)
    a = oracle.branch_sample(lg, [0, 500], u, 0.8)[0]
    b = oracle.branch_sample(lg * 2, [0, 500], u, 1.6)[0]
    assert np.array_equal(a, b)
    us = np.sort(u)
    assert np.all(np.diff(oracle.branch_sample(lg, [0, 500], us, 0.8)[0]) >= 0)


def test_branch_sample_matches_numpy_inverse_cdf_and_frequencies():
    rng = np.random.default_rng(4)
    S, V, T = 5, 64, 0.8
    lg = (rng.normal(size=(S, V)) * 2).astype(np.float32)
    pot = rng.integers(0, 4000, size=S)
    off = np.concatenate([[0], np.cumsum(pot)]).astype(np.int64)
    u = rng.random(int(off[-1])).astype(np.float32)
    tokens, seq, margin = oracle.branch_sample(lg, off, u, T)
    for s in range(S):
        p = np.exp((lg[s].astype(np.float64) - lg[s].max()) / T)
        cdf = np.cumsum(p)
        want = np.searchsorted(cdf, u[off[s]:off[s + 1]].astype(np.float64) * cdf[-1], side="right")
        got = tokens[off[s]:off[s + 1]]
        ok = margin[off[s]:off[s + 1]] > 1e-12
        assert np.array_equal(got[ok], want[ok]) and np.all(seq[off[s]:off[s + 1]] == s)
        if pot[s] > 2000:                                 # empirical frequencies follow the softmax
            freq = np.bincount(got, minlength=V) / pot[s]
            assert np.abs(freq - p / p.sum()).max() < 0.05


# =========================================================================================================
# gather of the unique paths' descriptor rows
# =========================================================================================================
def test_gather_unique_closed_forms_and_vectorised_second_way():
    rng = np.random.default_rng(77)
    # all paths unique: the gather is the identity and the offsets are the input offsets
    n = 9
    q_len = rng.integers(1, 6, size=n).astype(np.int32)
    q_off = np.concatenate([[0], np.cumsum(q_len)]).astype(np.int64)
    leaf = rng.permutation(n).astype(np.int32)
    g = oracle.gather_unique(np.arange(n, dtype=np.int32), n, n, leaf, q_len, q_off)
    assert np.array_equal(g["u_leaf"], leaf) and np.array_equal(g["u_q_len"], q_len)
    assert np.array_equal(g["u_q_offsets"], q_off) and np.array_equal(g["u_q_src"], q_off[:-1])
    # worked example of the paper (three equal samples and one different -> unique paths 0 and 3)
    g = oracle.gather_unique(np.asarray([0, 3, 0, 0], np.int32), 2, 4, np.asarray([10, 11, 12, 13], np.int32),
                             np.asarray([1, 1, 1, 1], np.int32), np.arange(5, dtype=np.int64))
    assert g["u_leaf"].tolist() == [10, 13, -1, -1] and g["u_q_len"].tolist() == [1, 1, 0, 0]
    assert g["u_q_offsets"].tolist() == [0, 1, 2, 2, 2] and g["u_q_src"].tolist() == [0, 3, 0, 0]
    # random subsets, written a second way with fancy indexing + cumsum
    for _ in range(20):
        n = int(rng.integers(1, 60))
        U = int(rng.integers(0, n + 1))
        uniq = np.sort(rng.choice(n, size=U, replace=False)).astype(np.int32)
        up = np.concatenate([uniq, rng.integers(0, n, size=n - U).astype(np.int32)])     # garbage past U
        q_len = rng.integers(0, 130, size=n).astype(np.int32)
        q_off = (np.concatenate([[0], np.cumsum(q_len)]) + 5).astype(np.int64)
        leaf = rng.integers(0, 1000, size=n).astype(np.int32)
        g = oracle.gather_unique(up, U, n, leaf, q_len, q_off)
        assert np.array_equal(g["u_leaf"][:U], leaf[uniq]) and np.all(g["u_leaf"][U:] == -1)
        assert np.array_equal(g["u_q_len"][:U], q_len[uniq]) and np.all(g["u_q_len"][U:] == 0)
        assert np.array_equal(g["u_q_src"][:U], q_off[uniq]) and np.all(g["u_q_src"][U:] == 0)
        want = np.concatenate([[0], np.cumsum(q_len[uniq].astype(np.int64))])
        assert np.array_equal(g["u_q_offsets"][:U + 1], want) and np.all(g["u_q_offsets"][U:] == want[-1])
    # empty batch
    g = oracle.gather_unique(np.zeros(0, np.int32), 0, 0, np.zeros(0, np.int32), np.zeros(0, np.int32),
                             np.zeros(1, np.int64))
    assert g["u_q_offsets"].tolist() == [0]


# =========================================================================================================
# radix tree over whole pages
# =========================================================================================================
def check_prefix_tree_invariants(seqs, t, page):
    """Properties that characterise the tree, checked without the oracle's algorithm."""
    n = len(seqs)
    order, leaf = t["order"], t["path_leaf_node"]
    parent, kv, sp, so = t["node_parent"], t["node_kv_len"], t["node_src_path"], t["node_src_offset"]
    assert sorted(order.tolist()) == list(range(n))
    keys = [(tuple(seqs[i]), i) for i in order]
    assert keys == sorted(keys)                                        # lexicographic, ties by index
    assert all(parent[v] < v for v in range(len(parent)))              # parents precede children
    below = [[] for _ in parent]
    for r in range(n):
        # the chain root -> leaf spells the path
        chain, v = [], int(leaf[r])
        while v >= 0:
            chain.append(v); v = int(parent[v])
        toks = []
        for v in reversed(chain):
            assert so[v] == len(toks)                                  # a node starts where the chain above it ends
            toks += list(seqs[sp[v]][so[v]:so[v] + kv[v]])
            below[v].append(r)
        assert toks == list(seqs[order[r]])
    children = [[] for _ in parent]
    for v in range(len(parent)):
        if parent[v] >= 0:
            children[parent[v]].append(v)
    n_inner = 0
    for v in range(len(parent)):
        b = below[v]
        assert b == list(range(b[0], b[-1] + 1))                       # the paths below a node are contiguous
        if len(b) > 1:
            n_inner += 1
            assert kv[v] % page == 0 and kv[v] > 0                     # shared nodes hold whole pages
            assert len(children[v]) >= 2                               # ... and branch
    assert n_inner + n == len(parent)                                  # everything else is a private leaf
    # maximality: two children of one parent (or two roots) never start with the same full page
    groups = {}
    for v in range(len(parent)):
        groups.setdefault(int(parent[v]), []).append(v)
    for vs in groups.values():
        firsts = [tuple(seqs[order[below[v][0]]][so[v]:so[v] + page]) for v in vs
                  if len(seqs[order[below[v][0]]]) - so[v] >= page]
        assert len(firsts) == len(set(firsts))


def test_prefix_tree_hand_worked_example():
    want = {}
    for line in open(os.path.join(GOLDEN, "prefix_tree_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        want[k] = [int(x) for x in v]
    seqs = [[1, 2, 3, 4, 5, 6, 7, 8, 9], [1, 2, 3, 4, 5, 6, 7, 8, 10, 11], [1, 2, 3, 4, 9, 9, 9, 9], [7],
            [1, 2, 3, 4, 5, 6, 7, 8], []]
    ids, off = csr(seqs)
    t = oracle.build_prefix_tree(ids, off, want["page_size"][0])
    for k in ("order", "path_leaf_node", "node_parent", "node_kv_len", "node_src_offset"):
        assert t[k].tolist() == want[k], k
    check_prefix_tree_invariants(seqs, t, 4)


@pytest.mark.parametrize("seed", range(12))
def test_prefix_tree_invariants_on_random_trees(seed):
    """Sequences drawn from a random tree with known sharing: the oracle's tree must spell every path, share whole
    pages only, be maximal, and share exactly as many tokens as the generating tree does."""
    rng = np.random.default_rng(seed)
    page = int(rng.choice([2, 4, 16]))
    seqs = []

    def grow(prefix, depth):
        fan = int(rng.integers(1, 4)) if depth < 3 else 1
        for _ in range(fan):
            if depth < 3 and rng.random() < 0.6:
                seg = [int(x) for x in rng.integers(0, 3, size=page * int(rng.integers(1, 3)))]
                grow(prefix + seg, depth + 1)
            else:
                seqs.append(prefix + [int(x) for x in rng.integers(0, 3, size=int(rng.integers(0, 2 * page)))])

    grow([], 0)
    perm = rng.permutation(len(seqs))
    seqs = [seqs[i] for i in perm]
    ids, off = csr(seqs)
    t = oracle.build_prefix_tree(ids, off, page)
    check_prefix_tree_invariants(seqs, t, page)
    # tokens stored = sum over sorted neighbours of what is NOT shared in whole pages (brute force, second way)
    order = t["order"]
    stored = len(seqs[order[0]]) if len(seqs) else 0
    for r in range(1, len(seqs)):
        a, b = seqs[order[r - 1]], seqs[order[r]]
        k = 0
        while k < len(a) and k < len(b) and a[k] == b[k]:
            k += 1
        stored += len(b) - (k // page) * page
    assert int(t["node_kv_len"].sum()) == stored
