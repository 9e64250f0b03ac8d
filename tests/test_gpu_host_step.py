"""ss_candidate_step_host: the whole path for host-resident per-step data, checked against the CPU oracle and against
the device-resident calls (same kernels, so the results must be bit-identical)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import binding as B
from paper_2609_39334_b200 import synth
from paper_2609_39334_b200.pipeline import DevicePipeline, HostStepPipeline
from test_gpu_parity import check_attention, check_dedup, check_topk

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_host_step_matches_oracle_and_device_path(cfg):
    w = synth.make_config(cfg)
    pipe = DevicePipeline(w, DEV, attn_flags=B.SS_FLAG_VALIDATE)
    pipe.step()
    r_dev = pipe.results()
    host = HostStepPipeline(pipe, depth=2)
    # poison the device-resident per-step inputs of `pipe`: the host call must not depend on them
    pipe.q.zero_()
    pipe.tok_ids.zero_()
    for i in range(4):                       # both sets, each twice, all in flight together
        host.submit(i)
    host.synchronize()
    for i in range(2):
        r = host.results(i)
        ref = check_dedup(r, w)
        check_topk(r, w)
        check_attention(r, w, ref, max_paths=24 if cfg != 3 else 8)
        for key in ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out", "survivors", "keep"):
            assert np.array_equal(r[key], r_dev[key]), key
        assert r["total_q"] == r_dev["total_q"]
        assert np.array_equal(r["out"], r_dev["out"])
        assert np.array_equal(r["lse"], r_dev["lse"])


def test_host_step_empty_batch_and_errors():
    w = synth.make_config(1)
    pipe = DevicePipeline(w, DEV)
    host = HostStepPipeline(pipe, depth=1)
    s = host.sets[0]
    # arena too small
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    assert B.ss_candidate_step_host(s["step"], small, check=False) == B.SS_ERR_WORKSPACE_TOO_SMALL
    # bad struct size
    good = s["step"].struct_size
    s["step"].struct_size = good - 8
    assert B.ss_candidate_step_host(s["step"], s["arena"], check=False) == B.SS_ERR_INVALID_ARG
    s["step"].struct_size = good
    # empty batch: only the counters are written
    s["step"].n_paths = 0
    s["step"].n_segments = 0
    s["step"].total_tok = 0
    s["step"].total_q = 0
    s["h_out"]["num_unique"].fill_(77)
    s["h_out"]["u_q_offsets"].fill_(77)
    B.ss_candidate_step_host(s["step"], s["arena"], stream=s["stream"])
    s["stream"].synchronize()
    assert int(s["h_out"]["num_unique"][0]) == 0 and int(s["h_out"]["u_q_offsets"][0]) == 0
    assert int(s["h_out"]["device_status"][0]) == B.SS_OK


@pytest.mark.parametrize("cfg", [2, 4])
def test_host_step_with_compact_transfers_returns_only_live_rows(cfg):
    """SS_STEP_COMPACT_TRANSFERS: only the live rows of out / lse come back (a duplicate gets no forward pass, hence no
    output of its own).  Rows past the live ones must stay as the caller left them, and the results equal those of the
    device-resident calls bit for bit."""
    w = synth.make_config(cfg)
    pipe = DevicePipeline(w, DEV)
    pipe.step()
    r_dev = pipe.results()
    host = HostStepPipeline(pipe, depth=2, compact=True)
    full_in, full_out = host.h2d_bytes, host.d2h_bytes
    assert host.measure_traffic()
    U, tq = r_dev["num_unique"], r_dev["total_q"]
    assert U < w.num_paths and tq < w.total_q
    row = w.num_q_heads * w.head_dim * 2
    assert host.h2d_bytes == full_in
    assert host.d2h_bytes == full_out - (w.total_q - tq) * (row + w.num_q_heads * 4)
    for i in range(4):
        host.submit(i)
    host.synchronize()
    for i in range(2):
        r = host.results(i)
        assert np.array_equal(r["out"], r_dev["out"]) and np.array_equal(r["lse"], r_dev["lse"])
        for key in ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out", "survivors", "keep"):
            assert np.array_equal(r[key], r_dev[key]), key
