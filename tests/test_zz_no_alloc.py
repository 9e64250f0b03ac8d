"""ss_dedup_paths_static: the deduplication entry point for callers that cannot allocate device memory (an engine
whose free HBM all belongs to its KV-cache pool, a loop that cannot take an allocator's synchronisation, a plug-in
without allocator rights).  Its scratch is a fixed array inside the library, so the only things the test hands over
are inputs and outputs; the results must be bit-identical to ss_dedup_paths with a caller workspace, on two calls
in a row (the second call finds the first call's leftovers in the shared scratch).

This file is collected last on purpose: a run that stops at the first failure has then already run every other
test."""
import numpy as np
import pytest
import torch

from paper_2609_39334_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(seed, n):
    rng = np.random.default_rng(seed)
    lens = rng.integers(0, 6, size=n)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    ids = rng.integers(0, 3, size=max(int(off[-1]), 1)).astype(np.int32)
    ctx = rng.integers(0, 2, size=n).astype(np.int64)
    slot = rng.integers(0, 1 << 20, size=n).astype(np.int32)
    return [torch.from_numpy(a).to(DEV) for a in (ids, off, ctx, slot)]


def _outputs(n):
    i32 = dict(dtype=torch.int32, device=DEV)
    return [torch.full((n,), -5, **i32) for _ in range(5)] + [torch.full((1,), -5, **i32)]


def _run(static, ids, off, ctx, slot, n):
    canon, p2u, uniq, mult, slot_out, nu = _outputs(n)
    if static:
        B.ss_dedup_paths_static(ids, off, ctx, slot, n, 0, canon, p2u, uniq, mult, slot_out, nu)
    else:
        ws = B.alloc_workspace(B.ss_dedup_workspace_bytes(n), DEV)
        B.ss_dedup_paths(ids, off, ctx, slot, n, 0, canon, p2u, uniq, mult, slot_out, nu, ws)
    torch.cuda.synchronize()
    u = int(nu.item())
    return u, canon.cpu(), p2u.cpu(), uniq[:u].cpu(), mult[:u].cpu(), slot_out.cpu()


def test_static_scratch_dedup_matches_workspace_dedup_twice_in_a_row():
    # two different batches back to back: the second one runs on a scratch array full of the first one's data
    for seed, n in [(1, 5000), (2, 777)]:
        ids, off, ctx, slot = _case(seed, n)
        want = _run(False, ids, off, ctx, slot, n)
        got = _run(True, ids, off, ctx, slot, n)
        assert got[0] == want[0] and 0 < got[0] < n
        for g, w in zip(got[1:], want[1:]):
            assert torch.equal(g, w)


def test_static_scratch_dedup_small_and_empty_batches():
    # batches of at most 4096 paths take the two-launch path and batches of up to 32768 the three-launch one: their
    # arrival counters live inside the shared scratch and
    # must start at zero on every call; n = 0 writes only the count
    for seed, n in [(3, 4096), (4, 300), (5, 1), (6, 4096), (8, 16384), (9, 16385)]:
        ids, off, ctx, slot = _case(seed, n)
        want = _run(False, ids, off, ctx, slot, n)
        got = _run(True, ids, off, ctx, slot, n)
        assert got[0] == want[0] and 0 < got[0] <= n
        for g, w in zip(got[1:], want[1:]):
            assert torch.equal(g, w)
    one = torch.zeros(1, dtype=torch.int32, device=DEV)
    off0 = torch.zeros(1, dtype=torch.int64, device=DEV)
    outs = _outputs(1)
    B.ss_dedup_paths_static(one, off0, None, None, 0, 0, outs[0], outs[1], outs[2], outs[3], None, outs[5])
    torch.cuda.synchronize()
    assert int(outs[5].item()) == 0
    assert all(int(o.item()) == -5 for o in outs[:4])      # nothing but the count was written


def test_static_scratch_dedup_at_its_maximum_and_without_allocating():
    n = B.SS_DEDUP_STATIC_MAX_PATHS
    ids, off, ctx, slot = _case(7, n)
    want = _run(False, ids, off, ctx, slot, n)
    got = _run(True, ids, off, ctx, slot, n)               # (also the warm call: the scratch address is now cached)
    assert got[0] == want[0]
    for g, w in zip(got[1:], want[1:]):
        assert torch.equal(g, w)
    # the property the entry point exists for: a call leaves the device's free memory and the framework's allocator
    # exactly as it found them
    canon, p2u, uniq, mult, slot_out, nu = _outputs(n)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    B.ss_dedup_paths_static(ids, off, ctx, slot, n, 0, canon, p2u, uniq, mult, slot_out, nu)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert int(nu.item()) == want[0]


def test_static_scratch_dedup_rejects_batches_beyond_its_maximum():
    n = B.SS_DEDUP_STATIC_MAX_PATHS + 1
    one = torch.zeros(1, dtype=torch.int32, device=DEV)
    off = torch.zeros(n + 1, dtype=torch.int64, device=DEV)
    outs = _outputs(n)
    rc = B.ss_dedup_paths_static(one, off, None, None, n, 0, outs[0], outs[1], outs[2], outs[3], None, outs[5],
                                 check=False)
    assert rc == B.SS_ERR_UNSUPPORTED
    assert int(outs[5].item()) == -5          # nothing was launched
