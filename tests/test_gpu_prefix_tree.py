"""ss_build_prefix_tree against the CPU oracle: every output is unique, so the comparison is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_tree(ids, off, page):
    n = len(off) - 1
    dev = torch.device(DEV)

    def t(a, dt):
        a = np.ascontiguousarray(a, dtype=dt)
        return torch.from_numpy(a).to(dev) if a.size else torch.zeros(1, dtype=torch.from_numpy(a).dtype, device=dev)
    i32 = dict(dtype=torch.int32, device=dev)
    order = torch.full((max(n, 1),), -7, **i32)
    leaf = torch.full((max(n, 1),), -7, **i32)
    cap = max(2 * n, 1)
    parent, kv, sp, so = (torch.full((cap,), -7, **i32) for _ in range(4))
    num = torch.full((1,), -7, **i32)
    total = int(off[-1])
    ws = B.alloc_workspace(B.ss_prefix_tree_workspace_bytes(n, total, page), dev)
    B.ss_build_prefix_tree(t(ids, np.int32), t(off, np.int64), n, total, page, order, leaf, parent, kv, sp, so, num, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_OK
    m = int(num.item())
    return dict(order=order[:n].cpu().numpy(), path_leaf_node=leaf[:n].cpu().numpy(), node_parent=parent[:m].cpu().numpy(),
                node_kv_len=kv[:m].cpu().numpy(), node_src_path=sp[:m].cpu().numpy(), node_src_offset=so[:m].cpu().numpy())


def check(ids, off, page):
    got = run_tree(ids, off, page)
    want = oracle.build_prefix_tree(ids, off, page)
    for k in want:
        assert np.array_equal(got[k], want[k]), k
    return got


def csr(seqs):
    off = np.zeros(len(seqs) + 1, np.int64)
    for i, s in enumerate(seqs):
        off[i + 1] = off[i] + len(s)
    return np.asarray([x for s in seqs for x in s], np.int32), off


def random_tree_seqs(rng, page, alphabet, fan_max, depth_max, seg_pages, tail_max):
    seqs = []

    def grow(prefix, depth):
        for _ in range(int(rng.integers(1, fan_max + 1))):
            if depth < depth_max and rng.random() < 0.6:
                seg = [int(x) for x in rng.integers(0, alphabet, size=page * int(rng.integers(1, seg_pages + 1)))]
                grow(prefix + seg, depth + 1)
            else:
                seqs.append(prefix + [int(x) for x in rng.integers(0, alphabet, size=int(rng.integers(0, tail_max + 1)))])
    grow([], 0)
    perm = rng.permutation(len(seqs))
    return [seqs[i] for i in perm]


def test_prefix_tree_paper_style_example_on_gpu():
    seqs = [[1, 2, 3, 4, 5, 6, 7, 8, 9], [1, 2, 3, 4, 5, 6, 7, 8, 10, 11], [1, 2, 3, 4, 9, 9, 9, 9], [7],
            [1, 2, 3, 4, 5, 6, 7, 8], []]
    got = check(*csr(seqs), 4)
    assert got["node_parent"].tolist() == [-1, -1, 1, 2, 2, 2, 1, -1]
    assert got["node_kv_len"].tolist() == [0, 4, 4, 0, 1, 2, 4, 1]


@pytest.mark.parametrize("seed", range(8))
def test_prefix_tree_random_trees(seed):
    rng = np.random.default_rng(100 + seed)
    page = int(rng.choice([2, 4, 16]))
    seqs = random_tree_seqs(rng, page, alphabet=3, fan_max=4, depth_max=4, seg_pages=3, tail_max=2 * page)
    check(*csr(seqs), page)


def test_prefix_tree_edge_cases():
    for n in (0, 1):
        ids, off = csr([[5, 6, 7]] * n)
        got = check(ids, off, 16)
        assert len(got["node_parent"]) == n
    check(*csr([[], [], []]), 16)                                   # only empty paths: three empty root leaves
    check(*csr([[3] * 40] * 5), 16)                                 # identical paths: 2 shared pages + 5 leaves of 8
    check(*csr([[1] * 16, [1] * 32, [1] * 48, [1] * 15]), 16)       # every path a prefix of the next
    check(*csr([[2] * (4 * k) for k in range(700)]), 4)              # ... 700 deep: intervals nested at one start rank
    rng0 = np.random.default_rng(4)
    stair = [[3] * (4 * int(k)) + [5] for k in rng0.integers(0, 300, size=900)]
    check(*csr(stair), 4)                                           # nested on both sides, many equal neighbours
    rng = np.random.default_rng(1)
    check(*csr([[int(x) for x in rng.integers(0, 50000, size=int(rng.integers(0, 70)))] for _ in range(300)]), 16)


def test_prefix_tree_many_paths_long_shared_prefix():
    """More paths than one sort block (merges across blocks) and a long common prefix (the comparator's hash search)."""
    rng = np.random.default_rng(9)
    page = 16
    prompt = [int(x) for x in rng.integers(0, 1000, size=64 * page)]
    seqs = []
    for p in range(40):                                             # 40 problems x ~130 candidates
        head = prompt[:page * int(rng.integers(8, 64))] + [int(x) for x in rng.integers(0, 1000, size=page)]
        for c in range(int(rng.integers(100, 160))):
            step = [int(x) for x in rng.integers(0, 4, size=int(rng.integers(1, 50)))]
            seqs.append(head + step)
    perm = rng.permutation(len(seqs))
    seqs = [seqs[i] for i in perm]
    assert len(seqs) > 4096
    got = check(*csr(seqs), page)
    # whole-page sharing pays: the tree stores far fewer tokens than the paths hold
    assert int(got["node_kv_len"].sum()) < 0.2 * sum(len(s) for s in seqs)


def test_prefix_tree_feeds_tree_attention():
    """End to end: token ids -> ss_build_prefix_tree -> KV pool laid out by the tree's nodes (shared pages stored once)
    -> ss_tree_attention; the result must match the CPU oracle evaluated on a FLAT layout in which every path owns all
    of its pages.  K/V of a token are a function of the token prefix up to it, as they are in a causal model."""
    rng = np.random.default_rng(21)
    page, Hq, Hkv, D = 16, 8, 2, 128
    tok = lambda k: [int(x) for x in rng.integers(0, 50, size=k)]
    seqs = []
    for _ in range(3):                                           # prompt -> branches -> candidates, as in a search step
        prompt = tok(page * int(rng.integers(12, 21)))
        for _ in range(3):
            branch = prompt + tok(page * int(rng.integers(2, 5)))
            seqs += [branch + tok(int(rng.integers(1, 71))) for _ in range(12)]
        seqs += [prompt + tok(int(rng.integers(1, 30))) for _ in range(2)]
    seqs += [tok(int(rng.integers(1, 90))) for _ in range(4)]    # candidates that share nothing
    seqs = [seqs[i] for i in rng.permutation(len(seqs))]
    n = len(seqs)
    ids, off = csr(seqs)
    T = np.asarray([1 if i % 3 else min(len(seqs[i]), int(rng.integers(2, 40))) for i in range(n)], np.int32)

    kv_cache = {}

    def kv_of(path):                                             # [len][2][Hkv][D] bf16, keyed by the running prefix
        h, rows = 1469598103934665603, []
        for tok in seqs[path]:
            h = ((h ^ (tok + 1)) * 1099511628211) % (1 << 64)
            if h not in kv_cache:
                kv_cache[h] = torch.from_numpy(np.random.default_rng(h % (1 << 32)).standard_normal((2, Hkv, D)).astype(np.float32)).to(torch.bfloat16)
            rows.append(kv_cache[h])
        return torch.stack(rows) if rows else torch.zeros((0, 2, Hkv, D), dtype=torch.bfloat16)

    def lay_out(node_tokens):
        """node_tokens: list of [len][2][Hkv][D] -> pool [pages][2][Hkv][16][D], page offsets, page ids."""
        offs, pages = [0], []
        for kv in node_tokens:
            offs.append(offs[-1] + (kv.shape[0] + page - 1) // page)
        pool = torch.zeros((max(offs[-1], 1), 2, Hkv, page, D), dtype=torch.bfloat16)
        for v, kv in enumerate(node_tokens):
            for t in range(kv.shape[0]):
                pool[offs[v] + t // page, :, :, t % page, :] = kv[t]
        return pool, np.asarray(offs, np.int64), np.arange(offs[-1], dtype=np.int32)

    per_path = [kv_of(i) for i in range(n)]
    q = torch.from_numpy(rng.standard_normal((int(T.sum()), Hq, D)).astype(np.float32)).to(torch.bfloat16)
    q_off = np.concatenate([[0], np.cumsum(T)]).astype(np.int64)

    # ---- reference: flat layout, CPU oracle ----------------------------------------------------------------------------
    pool_f, po_f, pg_f = lay_out(per_path)
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    pb = bits(pool_f)
    o_ref, l_ref = oracle.tree_attention(Hq, Hkv, D, page, 1.0 / np.sqrt(D), pb.reshape(-1), pb.reshape(-1)[Hkv * page * D:],
                                         2 * Hkv * page * D, page * D, D, np.full(n, -1, np.int32),
                                         np.asarray([len(s) for s in seqs], np.int32), po_f, pg_f,
                                         np.arange(n, dtype=np.int32), T, q_off, bits(q))

    # ---- tree layout from the GPU builder, GPU attention ---------------------------------------------------------------------
    t = run_tree(ids, off, page)
    want = oracle.build_prefix_tree(ids, off, page)
    for k in want:
        assert np.array_equal(t[k], want[k]), k
    node_tokens = [per_path[p][o:o + l] for p, o, l in zip(t["node_src_path"], t["node_src_offset"], t["node_kv_len"])]
    assert sum(x.shape[0] for x in node_tokens) < sum(len(s) for s in seqs)          # something is shared
    pool_t, po_t, pg_t = lay_out(node_tokens)
    order = t["order"]
    T_r = T[order]
    q_off_r = np.concatenate([[0], np.cumsum(T_r)]).astype(np.int64)
    q_r = torch.cat([q[q_off[i]:q_off[i + 1]] for i in order])
    dev = torch.device(DEV)
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    total_q = int(T.sum())
    out = torch.empty((total_q, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((total_q, Hq), dtype=torch.float32, device=dev)
    keep = [pool_t.to(dev), d(t["node_parent"]), d(t["node_kv_len"]), d(po_t), d(pg_t), d(t["path_leaf_node"]), d(T_r),
            d(q_off_r), q_r.to(dev)]
    desc = B.make_attn_desc(num_q_heads=Hq, num_kv_heads=Hkv, kv_pool=keep[0], node_parent=keep[1], node_kv_len=keep[2],
                            node_page_offsets=keep[3], node_pages=keep[4], total_node_pages=int(po_t[-1]),
                            path_leaf_node=keep[5], path_q_len=keep[6], q_offsets=keep[7], total_q=total_q, q=keep[8],
                            out=out, lse=lse, num_paths=n, flags=B.SS_FLAG_VALIDATE,
                            max_decode_paths=int((T == 1).sum()))
    ws = B.alloc_workspace(B.ss_tree_attention_workspace_bytes(desc), dev)
    B.ss_tree_attention(desc, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_OK
    got_o = out.to(torch.float64).cpu().numpy()
    got_l = lse.to(torch.float64).cpu().numpy()
    rows = np.concatenate([np.arange(q_off[i], q_off[i + 1]) for i in order])    # reference rows in rank order
    err = np.abs(got_o - o_ref[rows])
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.abs(got_l - l_ref[rows]).max() <= 1e-3
