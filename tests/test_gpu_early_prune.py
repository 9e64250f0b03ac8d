"""ss_early_prune on the GPU against the oracle: the paper's worked example, random partially-verified segments,
tie-heavy scores with many perfect ones, large segments, and agreement with ss_topk_prune once everything is verified."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run(scores, verified, seg, k):
    n, P = len(scores), len(seg) - 1
    dev = torch.device(DEV)
    sc = torch.from_numpy(np.ascontiguousarray(scores if n else np.zeros(1, np.float32), dtype=np.float32)).to(dev)
    ve = torch.from_numpy(np.ascontiguousarray(verified if n else np.zeros(1, np.uint8), dtype=np.uint8)).to(dev)
    sg = torch.from_numpy(np.ascontiguousarray(seg, dtype=np.int32)).to(dev)
    pruned = torch.full((max(n, 1),), 9, dtype=torch.uint8, device=dev)
    sel = torch.full((max(P, 1), k), -9, dtype=torch.int32, device=dev)
    fin = torch.full((max(P, 1),), 9, dtype=torch.uint8, device=dev)
    ws = B.alloc_workspace(B.ss_topk_workspace_bytes(n), dev)
    B.ss_early_prune(sc, ve, sg, P, n, k, pruned, sel, fin, ws)
    torch.cuda.synchronize()
    return pruned[:n].cpu().numpy(), sel[:P].cpu().numpy(), fin[:P].cpu().numpy()


def test_paper_worked_example_on_gpu():
    lines = [l.strip() for l in open(os.path.join(GOLDEN, "early_pruning_example.txt")) if l.strip() and not l.startswith("#")]
    k = int(lines[0].split()[1])
    names = lines[1].split()[1:]
    scores = np.zeros(len(names), np.float32)
    verified = np.zeros(len(names), np.uint8)
    seen = set()
    for line in lines[2:]:
        ev, pr, se = [x.strip() for x in line.split("|")]
        _, who, val = ev.split()
        scores[names.index(who)], verified[names.index(who)] = float(val), 1
        pruned, sel, fin = run(scores, verified, [0, len(names)], k)
        seen |= {names[i] for i in range(len(names)) if pruned[i]}
        want = set() if pr.split(":")[1].strip() == "-" else set(pr.split(":")[1].split())
        assert seen == want
        want_sel = se.split(":")[1].strip()
        assert (fin[0] == 0 and list(sel[0]) == [-1] * k) if want_sel == "-" else [names[i] for i in sel[0]] == want_sel.split()


@pytest.mark.parametrize("sizes,k", [([32] * 8, 8), ([0, 5, 0, 1, 70], 4), ([4096], 64), ([5000, 3, 9000], 100), ([7], 16),
                                     ([256] * 64, 64)])
def test_early_prune_vs_oracle(sizes, k):
    rng = np.random.default_rng(sum(sizes) * 7 + k)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    n = int(seg[-1])
    for perfect_frac in (0.0, 0.05, 0.4):
        sc = (rng.integers(0, 9, size=n) / 8.0).astype(np.float32) * np.float32(0.99)
        sc[rng.random(n) < perfect_frac] = 1.0
        for frac in (0.0, 0.2, 0.6, 1.0):
            ver = (rng.random(n) < frac).astype(np.uint8) if frac < 1.0 else np.ones(n, np.uint8)
            got = run(sc, ver, seg, k)
            want = oracle.early_prune(sc, ver, seg, k)
            for g, w in zip(got, want):
                assert np.array_equal(g, w)


def test_all_verified_agrees_with_topk_prune():
    rng = np.random.default_rng(11)
    seg = np.asarray([0, 40, 100, 164], np.int32)
    sc = (rng.random(164) * 0.9).astype(np.float32)
    pruned, sel, fin = run(sc, np.ones(164, np.uint8), seg, 8)
    surv, keep = oracle.topk(sc, seg, 8)
    assert fin.all() and np.array_equal(sel, surv) and np.array_equal(1 - pruned, keep)


def test_topk_and_early_prune_report_segments_outside_the_candidates():
    """Segment offsets index keep[] / pruned[] and the scratch region: a segment that does not lie inside [0, n_total]
    is reported through the status word and treated as empty, never followed."""
    dev = torch.device(DEV)
    n, k = 40, 3
    scores = torch.rand(n, device=dev)
    seg = torch.tensor([0, 10, 25, 4000], dtype=torch.int32, device=dev)      # the last segment runs past n
    surv = torch.full((3, k), -9, dtype=torch.int32, device=dev)
    keep = torch.full((n,), 7, dtype=torch.uint8, device=dev)
    ws = B.alloc_workspace(B.ss_topk_workspace_bytes(n), dev)
    B.ss_topk_prune(scores, seg, 3, n, k, surv, keep, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_ERR_BAD_INPUT
    assert surv[2].tolist() == [-1] * k and keep[25:].sum().item() == 0      # the bad segment selected nothing
    s_ref, k_ref = oracle.topk(scores.cpu().numpy(), np.asarray([0, 10, 25], np.int32), k)
    assert np.array_equal(surv[:2].cpu().numpy(), s_ref) and np.array_equal(keep[:25].cpu().numpy(), k_ref[:25])
    ver = torch.ones(n, dtype=torch.uint8, device=dev)
    pruned = torch.empty(n, dtype=torch.uint8, device=dev)
    sel = torch.empty((3, k), dtype=torch.int32, device=dev)
    fin = torch.empty(3, dtype=torch.uint8, device=dev)
    seg_bad = torch.tensor([0, 10, 5, 40], dtype=torch.int32, device=dev)     # not monotone
    B.ss_early_prune(scores, ver, seg_bad, 3, n, k, pruned, sel, fin, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_ERR_BAD_INPUT
    # a clean call clears the word again
    B.ss_topk_prune(scores, torch.tensor([0, 10, 25, 40], dtype=torch.int32, device=dev), 3, n, k, surv, keep, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_OK
