"""ss_branch_sample (+ grouping with ss_dedup_paths) on the GPU against the oracle."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run(logits, off, u, T):
    dev = torch.device(DEV)
    n = int(off[-1])
    lg = torch.from_numpy(np.ascontiguousarray(logits, dtype=np.float32)).to(dev)
    of = torch.from_numpy(np.ascontiguousarray(off, dtype=np.int64)).to(dev)
    un = torch.from_numpy(np.ascontiguousarray(u if n else np.zeros(1, np.float32), dtype=np.float32)).to(dev)
    tok = torch.full((max(n, 1),), -3, dtype=torch.int32, device=dev)
    seq = torch.full((max(n, 1),), -3, dtype=torch.int64, device=dev)
    B.ss_branch_sample(lg, of, un, logits.shape[0], logits.shape[1], T, tok, seq)
    torch.cuda.synchronize()
    return tok[:n], seq[:n]


def group(tok, seq):
    """Grouping of the draws with the library's own dedup: children and their potential sizes."""
    n = tok.numel()
    dev = tok.device
    i32 = dict(dtype=torch.int32, device=dev)
    outs = [torch.empty(n, **i32) for _ in range(4)]
    nu = torch.zeros(1, **i32)
    ws = B.alloc_workspace(B.ss_dedup_workspace_bytes(n), dev)
    B.ss_dedup_paths(tok.contiguous(), torch.arange(n + 1, dtype=torch.int64, device=dev), seq.contiguous(), None, n, 0,
                     outs[0], outs[1], outs[2], outs[3], None, nu, ws)
    torch.cuda.synchronize()
    U = int(nu.item())
    return outs[2][:U].cpu().numpy(), outs[3][:U].cpu().numpy()


def test_paper_worked_example_on_gpu():
    kv = {}
    for l in open(os.path.join(GOLDEN, "branch_sampling_example.txt")):
        if l.strip() and not l.startswith("#"):
            k, *v = l.split()
            kv[k] = v
    with np.errstate(divide="ignore"):
        logits = np.log(np.asarray([float(x) for x in kv["probs"]])).astype(np.float32)[None, :]
    u = np.asarray([float(x) for x in kv["uniforms"]], np.float32)
    tok, seq = run(logits, [0, len(u)], u, float(kv["temperature"][0]))
    assert tok.cpu().tolist() == [int(x) for x in kv["tokens"]]
    uniq, mult = group(tok, seq)
    assert mult.tolist() == [int(x) for x in kv["potentials"]]


@pytest.mark.parametrize("S,V,T,maxpot", [(3, 6, 1.0, 5), (16, 1000, 0.8, 40), (8, 4097, 1.3, 8), (4, 151936, 0.8, 32),
                                          (2, 151936, 0.8, 3000), (64, 32000, 0.5, 16)])
def test_branch_sample_vs_oracle(S, V, T, maxpot):
    rng = np.random.default_rng(S * 1000 + V)
    logits = (rng.normal(size=(S, V)) * 3).astype(np.float32)
    logits[rng.random((S, V)) < 0.01] = -np.inf                 # masked tokens
    pot = rng.integers(0, maxpot + 1, size=S)
    off = np.concatenate([[0], np.cumsum(pot)]).astype(np.int64)
    u = rng.random(int(off[-1])).astype(np.float32)
    tok, seq = run(logits, off, u, T)
    want_tok, want_seq, margin = oracle.branch_sample(logits, off, u, T)
    got = tok.cpu().numpy()
    assert np.array_equal(seq.cpu().numpy(), want_seq)
    sure = margin > 1e-12                                       # both sides decide in fp64
    assert np.array_equal(got[sure], want_tok[sure])
    # grouping: children and potential sizes equal the oracle's dedup of the oracle's draws
    if len(got) and sure.all():
        uniq, mult = group(tok, seq)
        r = oracle.dedup(want_tok, np.arange(len(want_tok) + 1), ctx_key=want_seq)
        assert np.array_equal(uniq, r["unique_paths"]) and np.array_equal(mult, r["multiplicity"])
        assert int(mult.sum()) == int(off[-1])
