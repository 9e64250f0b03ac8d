"""The N > 1 path of the benchmark on CPU: two gloo ranks build their own replicas (same shapes, different
problems), time a fake step, and agree on the max-over-ranks time and the whole-job rate."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_39334_b200 import replicas, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = replicas.replica_workload(synth.make_config, 2, rank, scale=1 / 16)
    dist.barrier()
    fake_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = replicas.max_over_ranks(fake_ms)
    rate = replicas.whole_job_rate(int(w.path_q_len.sum()), slowest)
    sig = int(np.int64(w.tok_ids[:64].astype(np.int64).sum()))
    out.put((rank, w.num_paths, int(w.node_kv_len[0]), sig, slowest, rate))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_run_disjoint_replicas_and_take_the_max_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, n0, len0, sig0, slow0, rate0), (r1, n1, len1, sig1, slow1, rate1) = res
    assert (r0, r1) == (0, 1)
    assert n0 == n1 == 64 and len0 == len1 == 512     # same shapes
    assert sig0 != sig1                               # different problems
    assert slow0 == slow1 == 15.0                     # max over ranks
    assert rate0 == rate1 == 2 * 64 / 15e-3           # whole-job units / slowest time


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(100, 10.0) == 100 / 10e-3
