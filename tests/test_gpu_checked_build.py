"""The checked build of the library (-DSS_CHECKED -> libspecscale_checked.so): range predicates compiled into the
kernels' own address arithmetic (page ids against the pool, partial slots against the workspace capacity, query and
output rows against the tensors).  It stands in for a memory checker: benchmark configurations 1-4 must run through it
with a clean status word and the same results as the oracle, and an out-of-range page id - which the production
build would follow - must come back as SS_ERR_BAD_INPUT with the access clamped, not executed.

The library is selected by SS_LIB_SUFFIX when the binding is imported, so the checked runs happen in a child process.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def child():
    import numpy as np
    import torch

    import oracle
    from paper_2609_39334_b200 import binding as B
    from paper_2609_39334_b200 import synth
    from paper_2609_39334_b200.pipeline import DevicePipeline

    assert B.LIB_PATH.endswith("_checked.so")
    dev = "cuda:0"
    for cfg in (1, 2, 3, 4):
        w = synth.make_config(cfg, scale=0.5 if cfg == 3 else 1.0)
        pipe = DevicePipeline(w, dev)                     # no SS_FLAG_VALIDATE: the kernels' own checks are under test
        pipe.step()
        r = pipe.results()                                # raises unless the status word is clean
        ref = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
        assert r["num_unique"] == ref["num_unique"] and np.array_equal(r["unique_paths"], ref["unique_paths"])
        uniq = ref["unique_paths"][:: max(1, ref["num_unique"] // 24)]
        o_ref, l_ref = oracle.tree_attention_workload(w, paths=uniq)
        T = w.path_q_len[ref["unique_paths"]].astype(np.int64)
        off = np.concatenate([[0], np.cumsum(T)])
        pos = {int(u): i for i, u in enumerate(ref["unique_paths"])}
        rows = np.concatenate([np.arange(off[pos[int(u)]], off[pos[int(u)] + 1]) for u in uniq])
        err = np.abs(r["out"][rows] - o_ref)
        fin = np.isfinite(l_ref)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (cfg, err.max(), err.mean())
        assert np.abs(r["lse"][rows][fin] - l_ref[fin]).max() <= 1e-3
        print(f"checked build: config {cfg} ok ({len(uniq)} paths compared)")
    # a page table that points past the pool: refused by the predicates, the bad id is never used as an address
    w = synth.build_tree_workload("badpage", 11, 8, 2, [64], [6], 2, (20, 90), lambda i, n, rng: 1 + (i % 2) * 20)
    w.node_pages = w.node_pages.copy()
    w.node_pages[-1] = w.num_pages + 5
    w.node_pages[0] = -3
    pipe = DevicePipeline(w, dev)
    pipe.step()
    torch.cuda.synchronize()
    assert B.ss_last_device_status(pipe.attn_ws) == B.SS_ERR_BAD_INPUT
    print("checked build: out-of-range page id reported")


def test_checked_build_runs_the_benchmark_configurations_clean_and_refuses_a_bad_page_id():
    from paper_2609_39334_b200 import build as cuda_build
    cuda_build.build(defines=["SS_CHECKED"], suffix="_checked")
    env = dict(os.environ, SS_LIB_SUFFIX="_checked", PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    p = subprocess.run([sys.executable, os.path.abspath(__file__), "--child"], env=env, capture_output=True, text=True,
                       timeout=900)
    assert p.returncode == 0, p.stdout[-2000:] + p.stderr[-4000:]
    assert "config 4 ok" in p.stdout and "out-of-range page id reported" in p.stdout


if __name__ == "__main__" and "--child" in sys.argv:
    child()
