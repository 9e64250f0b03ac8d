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
