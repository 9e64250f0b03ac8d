#!/usr/bin/env python
"""Benchmark of the candidate-path hot path: one step = ss_dedup_paths -> gather of the unique paths ->
ss_tree_attention -> ss_topk_prune over one batch of seeded synthetic candidate trees.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5] [--impl reference]

Prints ONE JSON line.  metric = candidate-path query tokens/s (query tokens of all N logical candidates divided
by the step time).  `value` has every input resident in HBM; `e2e` copies the step's inputs from pinned host
memory and reads the results back inside the timed region.  `roofline` is for the dominant attention kernel,
timed live with CUDA events on the launching stream.  `cpu_baseline` is the CPU oracle on a bounded sample.
With --impl reference the CPU oracle is the timed arm.  Under torchrun every rank runs its own replica of the
workload (disjoint problems, no collective on the data path; weak scaling).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate_path_query_tokens_per_s"
UNIT = "tokens/s"
WORKLOADS = {"c2": 2, "c3": 3, "c4": 4, "c5": 5}
LV_SWEEP_TOKENS = [256, 512, 1024, 2048, 4096, 8192, 16384]
L2_BYTES = 126 * 1024 * 1024
MIN_ORACLE_SAMPLE = 128             # unique paths in the oracle's bounded sample
NOMINAL_HBM_GBS = 8000.0            # vendor figures, reported beside the measured peaks for context only
NOMINAL_BF16_TFLOPS = 2250.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------------------
# algorithmic work of one step (what the method must do; computed from the tree and the unique set)
# ------------------------------------------------------------------------------------------------------------
def algorithmic_work(w, unique_paths):
    """-> dict(tile_flops, leaf_bytes, unique_kv_bytes, tokens).  flops = 4*D per unmasked (query row, key) pair
    of the rows that run on the tensor-core tiles (shared nodes of decode paths, whole chain of verification
    paths); leaf bytes = K+V bytes of the private leaves of unique decode paths, read once."""
    D, Hq, Hkv = w.head_dim, w.num_q_heads, w.num_kv_heads
    kv_token_bytes = 2 * Hkv * D * 2
    node_start = np.zeros(w.num_nodes, np.int64)
    for n in range(w.num_nodes):
        p = int(w.node_parent[n])
        node_start[n] = 0 if p < 0 else node_start[p] + int(w.node_kv_len[p])
    leaf = w.path_leaf_node[unique_paths]
    T = w.path_q_len[unique_paths].astype(np.int64)
    leaf_len = w.node_kv_len[leaf].astype(np.int64)
    prefix_len = node_start[leaf]
    L = prefix_len + leaf_len
    dec = T == 1
    pairs_dec_shared = int(prefix_len[dec].sum())
    # verification: sum_t (L - T + t + 1) = T*L - T*(T-1)/2
    Tv, Lv = T[~dec], L[~dec]
    pairs_ver = int((Tv * Lv - Tv * (Tv - 1) // 2).sum())
    tile_flops = 4.0 * D * Hq * (pairs_dec_shared + pairs_ver)
    leaf_bytes = float(leaf_len[dec].sum()) * kv_token_bytes
    used_nodes = np.zeros(w.num_nodes, bool)
    for l in np.unique(leaf):
        n = int(l)
        while n >= 0 and not used_nodes[n]:
            used_nodes[n] = True
            n = int(w.node_parent[n])
    unique_kv_bytes = float(w.node_kv_len[used_nodes].astype(np.int64).sum()) * kv_token_bytes
    return dict(tile_flops=tile_flops, leaf_bytes=leaf_bytes, unique_kv_bytes=unique_kv_bytes,
                tokens=int(w.path_q_len.astype(np.int64).sum()))


# ------------------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()          # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, smax, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                smax.append(float(r[2]))
            except ValueError:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if r[col].lower() == "active":
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


# ------------------------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------------------
def oracle_sample(w, seed=0, budget_scale=1.0, min_paths=None):
    """A bounded sample of the workload for the CPU oracle: a few verification paths and more decode paths,
    sized by the host core count for roughly 10-30 s of CPU work per pass (`budget_scale` shrinks that for a run of
    many passes; `min_paths`: the least number of unique paths, MIN_ORACLE_SAMPLE unless given)."""
    if min_paths is None:
        min_paths = MIN_ORACLE_SAMPLE
    import oracle
    cores = oracle.host_cores()
    rng = np.random.default_rng(seed)
    ded = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
    uniq = ded["unique_paths"]
    T = w.path_q_len[uniq]
    ver, dec = uniq[T > 1], uniq[T == 1]
    # fp64 cost model: pairs * Hq * 2 * D multiply-adds; ~0.7 G mul-add/s per core for this plain loop
    budget_pairs = budget_scale * 12.0 * cores * 0.7e9 / (2.0 * w.head_dim * w.num_q_heads)
    chosen, pairs = [], 0.0
    pools = [list(rng.permutation(ver)), list(rng.permutation(dec))]
    turn = 0
    # one verification path, then three decode paths (a decode path costs 1/T of a verification path), until the
    # budget is spent AND at least MIN_ORACLE_SAMPLE unique paths are in
    while (pools[0] or pools[1]) and (pairs < budget_pairs or len(chosen) < min_paths):
        pool = pools[0] if (turn % 4 == 0 and pools[0]) or not pools[1] else pools[1]
        turn += 1
        p = int(pool.pop())
        pairs += int(w.path_q_len[p]) * w.path_kv_len(p)
        chosen.append(p)
    return np.asarray(sorted(chosen), np.int64)


def time_oracle(w_host, steps, warmup):
    import oracle
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        oracle.dedup(w_host.tok_ids, w_host.tok_offsets, w_host.ctx_key, w_host.slot_in)
        oracle.tree_attention_workload(w_host, paths=np.arange(w_host.num_paths))
        oracle.topk(w_host.scores, w_host.seg_offsets, w_host.top_k)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    return float(np.mean(times))


# ------------------------------------------------------------------------------------------------------------
# the smaller benchmark configurations and the "next" rows, reported inside the default run's JSON line
# ------------------------------------------------------------------------------------------------------------
class L2Flush:
    """Evicts L2 between timed iterations: a buffer of twice the L2 size is written, then a second one is read, so that
    the cache ends up full of CLEAN lines of data the step never touches.  (After a write alone, half of the buffer
    sits in L2 as dirty lines, and the step under test pays for their write-back: 126 MB of extra DRAM traffic inside
    the timed region, half as much again as a small configuration reads.)"""
    NOTE = "L2 flushed between iterations (252 MB written, then 252 MB read: no dirty lines left)"

    def __init__(self, dev):
        import torch
        self.w = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device=dev)
        self.sink = torch.zeros((), dtype=torch.int64, device=dev)

    def fill_(self, i):
        import torch
        self.w.fill_(i & 0xff)
        torch.sum(self.r, dim=(0,), out=self.sink)


def timed_ms(fn, steps, flush, dev):
    """CUDA-event time of `fn` per call, `steps` calls, L2 evicted before each (outside the events)."""
    import torch
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i, (a, b) in enumerate(ev):
        if flush is not None:
            flush.fill_(i & 0xff)
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize(dev)
    return [a.elapsed_time(b) for a, b in ev]


def small_workload(name, dev, flush, peaks, steps=20, warmup=5):
    """One of c2 / c3 / c4 (each well under a millisecond per step): whole step, attention call alone, per-phase
    times (the library's event profiler) and the two roofline fractions, with the clocks sampled meanwhile."""
    import torch
    from paper_2609_39334_b200 import binding as B
    from paper_2609_39334_b200 import synth
    from paper_2609_39334_b200.pipeline import DevicePipeline
    w = synth.make_config(WORKLOADS[name], device=dev, poison=True)
    pipe = DevicePipeline(w, dev)
    for _ in range(warmup):
        pipe.step()
    torch.cuda.synchronize(dev)
    st = B.ss_last_device_status(pipe.attn_ws)
    if st != B.SS_OK:
        raise B.SpecScaleError(st, f"{name} warm-up")
    clocks = ClockSampler(dev.index or 0)
    clocks.start()
    time.sleep(0.12)
    launches0 = B.ss_launch_count()
    step_ms = timed_ms(pipe.step, steps, flush, dev)
    launches = (B.ss_launch_count() - launches0) // steps
    attn_ms = timed_ms(pipe.attention, steps, flush, dev)
    B.ss_profile_read()
    B.ss_profile_enable(True)
    timed_ms(pipe.attention, steps, flush, dev)
    B.ss_profile_enable(False)
    phase_ms, phase_calls = B.ss_profile_read()
    time.sleep(0.12)
    clk = clocks.stop()
    st = B.ss_last_device_status(pipe.attn_ws)
    if st != B.SS_OK:
        raise B.SpecScaleError(st, name)
    U = int(pipe.num_unique.item())
    work = algorithmic_work(w, pipe.unique_paths[:U].cpu().numpy())
    tokens = work["tokens"]
    phases = {k: (phase_ms[k] / phase_calls[k] if phase_calls[k] else 0.0) for k in phase_ms}
    out = {"paths": w.num_paths, "unique_paths": U, "query_tokens": tokens,
           "heads": f"{w.num_q_heads}q/{w.num_kv_heads}kv", "launches_per_step": int(launches),
           "step_ms_median": float(np.median(step_ms)), "step_ms_min": float(min(step_ms)),
           "tokens_per_s": tokens / (float(np.median(step_ms)) * 1e-3),
           "attention_ms_median": float(np.median(attn_ms)), "attention_ms_min": float(min(attn_ms)),
           "attention_tokens_per_s": tokens / (float(np.median(attn_ms)) * 1e-3),
           "phase_ms": phases,
           "phase_note": "phase times carry the profiler's events (a few microseconds each); the attention and step "
                         "times above are measured without them",
           "l2": L2Flush.NOTE, "steps": steps, "warmup": warmup, "clocks": clk}
    if phases.get("tiles"):
        ach = work["tile_flops"] / (phases["tiles"] * 1e-3) / 1e12
        out["tiles"] = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_burst"], "unit": "TFLOP/s",
                        "frac": ach / peaks["bf16_burst"], "peak_kind": f"{peaks['source']} burst"}
    if phases.get("leaves") and work["leaf_bytes"] > 0:
        ach = work["leaf_bytes"] / (phases["leaves"] * 1e-3) / 1e9
        out["leaves"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": ach / peaks["hbm_gbs"], "peak_kind": f"{peaks['source']} copy",
                         "note": "the leaf launch also merges the partial results and writes the final rows"}
    hbm_s = work["unique_kv_bytes"] / (peaks["hbm_gbs"] * 1e9)
    tensor_s = work["tile_flops"] / (peaks["bf16_burst"] * 1e12)
    out["attention_roofline_ms"] = 1e3 * max(hbm_s, tensor_s)
    out["attention_frac_of_roofline"] = out["attention_roofline_ms"] / out["attention_ms_median"]
    del pipe, w
    torch.cuda.empty_cache()
    return out


def next_rows(dev, flush, peaks, steps=20):
    """Numbers for the rows beyond the core path: on-demand branching draws, radix-tree construction, early pruning
    with partially verified candidates, and the knee of the verification-batch curve."""
    import torch
    from paper_2609_39334_b200 import binding as B
    rng = np.random.default_rng(12345)
    out = {}
    # ---- ss_branch_sample: c2-shaped expansion (922 sequences drawing ~1024 candidates from 151936-token rows) --------
    S, V = 922, 151936
    logits = torch.randn((S, V), dtype=torch.float32, device=dev) * 3
    pot = rng.integers(1, 3, size=S)
    off = torch.from_numpy(np.concatenate([[0], np.cumsum(pot)]).astype(np.int64)).to(dev)
    n = int(pot.sum())
    u = torch.from_numpy(rng.random(n).astype(np.float32)).to(dev)
    tok = torch.empty(n, dtype=torch.int32, device=dev)
    seq = torch.empty(n, dtype=torch.int64, device=dev)
    fn = lambda: B.ss_branch_sample(logits, off, u, S, V, 0.8, tok, seq)
    fn()
    ms = float(np.median(timed_ms(fn, steps, flush, dev)))
    gbs = S * V * 4 / (ms * 1e-3) / 1e9
    out["ss_branch_sample"] = {"sequences": S, "vocab": V, "draws": n, "ms": ms, "logit_gb_per_s": gbs,
                               "frac_of_hbm": gbs / peaks["hbm_gbs"], "algorithmic_bytes": "4 B per logit, read once"}
    del logits
    # ---- ss_build_prefix_tree: c5-shaped ids (64 prompts of 4096 tokens x 256 candidates with 128-1024 own tokens) ----
    P_, F_ = 64, 256
    lens = rng.integers(128, 1025, size=P_ * F_) + 4096
    off_np = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    total = int(off_np[-1])
    ids = torch.randint(0, 151936, (total,), dtype=torch.int32, device=dev)
    off_t = torch.from_numpy(off_np).to(dev)
    prompts = torch.randint(0, 151936, (P_, 4096), dtype=torch.int32, device=dev)
    starts = off_t[:-1]
    idx = (starts[:, None] + torch.arange(4096, device=dev)[None, :]).reshape(-1)
    ids[idx] = prompts.repeat_interleave(F_, dim=0).reshape(-1)
    del idx, prompts
    npaths = P_ * F_
    i32 = dict(dtype=torch.int32, device=dev)
    order, leaf = torch.empty(npaths, **i32), torch.empty(npaths, **i32)
    parent, kv, sp, so = (torch.empty(2 * npaths, **i32) for _ in range(4))
    num = torch.zeros(1, **i32)
    ws = B.alloc_workspace(B.ss_prefix_tree_workspace_bytes(npaths, total, 16), dev)
    fn = lambda: B.ss_build_prefix_tree(ids, off_t, npaths, total, 16, order, leaf, parent, kv, sp, so, num, ws)
    fn()
    ms = float(np.median(timed_ms(fn, max(steps // 4, 3), None, dev)))
    out["ss_build_prefix_tree"] = {"paths": npaths, "token_ids": total, "nodes": int(num.item()), "ms": ms,
                                   "id_gb_per_s": total * 4 / (ms * 1e-3) / 1e9,
                                   "status": B.ss_last_device_status(ws)}
    del ids, ws
    # ---- ss_early_prune: c5-shaped segments (64 problems x 256 candidates, half of them verified, k = 64) ----------------
    n = 16384
    scores = torch.from_numpy(np.round(rng.random(n) * 8).astype(np.float32) / 8).to(dev)
    verified = torch.from_numpy((rng.random(n) < 0.5).astype(np.uint8)).to(dev)
    seg = torch.arange(0, n + 1, 256, dtype=torch.int32, device=dev)
    pruned = torch.empty(n, dtype=torch.uint8, device=dev)
    selected = torch.empty((64, 64), **i32)
    final = torch.empty(64, dtype=torch.uint8, device=dev)
    ws = B.alloc_workspace(B.ss_topk_workspace_bytes(n), dev)
    fn = lambda: B.ss_early_prune(scores, verified, seg, 64, n, 64, pruned, selected, final, ws)
    fn()
    out["ss_early_prune"] = {"candidates": n, "segments": 64, "k": 64,
                             "ms": float(np.median(timed_ms(fn, steps, flush, dev)))}
    torch.cuda.empty_cache()
    return out


def lv_curve(dev, flush, steps, warmup):
    """Verification-attention throughput against the number of batched step tokens (see lv_sweep)."""
    import torch
    from paper_2609_39334_b200 import binding as B
    from paper_2609_39334_b200 import synth
    from paper_2609_39334_b200.pipeline import DevicePipeline
    curve = []
    for target in LV_SWEEP_TOKENS:
        problems = max(1, target // (8 * 72))
        per = max(1, round(target / (72 * problems)))
        w = synth.build_tree_workload(f"lv{target}", synth.BASE_SEED + 100 + target, 28, 4, [1024], [per], problems,
                                      (64, 512), lambda i, n, rng: int(rng.integers(16, 129)), device=dev)
        pipe = DevicePipeline(w, dev)
        pipe.dedup()
        pipe.compact_unique()
        for _ in range(max(warmup, 3)):
            pipe.attention()
        torch.cuda.synchronize(dev)
        ms = float(np.median(timed_ms(pipe.attention, steps, flush, dev)))
        st = B.ss_last_device_status(pipe.attn_ws)
        if st != B.SS_OK:
            raise B.SpecScaleError(st, "lv-sweep")
        tokens = int(w.path_q_len.sum())
        curve.append({"batched_tokens": tokens, "candidates": w.num_paths, "ms": ms, "tokens_per_s": tokens / (ms * 1e-3)})
        del pipe, w
    # knee: the smallest batch that reaches 90 % of the largest batch's tokens/s (linear interpolation between points)
    top = curve[-1]["tokens_per_s"]
    knee = None
    for a, b in zip(curve, curve[1:]):
        if a["tokens_per_s"] < 0.9 * top <= b["tokens_per_s"]:
            f = (0.9 * top - a["tokens_per_s"]) / (b["tokens_per_s"] - a["tokens_per_s"])
            knee = a["batched_tokens"] + f * (b["batched_tokens"] - a["batched_tokens"])
    if knee is None and curve[0]["tokens_per_s"] >= 0.9 * top:
        knee = curve[0]["batched_tokens"]
    return curve, knee


def lv_sweep(args):
    """Attention-only analogue of the paper's verification-throughput profile (Section "Lazy Verification": the
    token threshold of the first flush policy is read off a throughput-vs-batched-tokens curve).  For each batch
    size a set of verification steps (7B reward-model head shape, 1024-token prompt, 64-512 prior tokens, steps of
    16-128 tokens, 8 candidates per problem) is attended in one ss_tree_attention call; reported is step tokens/s."""
    import torch
    from paper_2609_39334_b200 import binding as B
    from paper_2609_39334_b200 import synth
    from paper_2609_39334_b200.pipeline import DevicePipeline
    assert torch.cuda.is_available(), "bench.py needs a GPU (there is no CPU fallback)"
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    if int(os.environ.get("RANK", "0")) != 0:
        return
    flush = L2Flush(dev)
    curve, knee = lv_curve(dev, flush, args.steps, args.warmup)
    print(json.dumps({"metric": "verification_attention_step_tokens_per_s", "unit": "tokens/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "lv-sweep", "heads": "28q/4kv", "prefix": 1024, "l2": L2Flush.NOTE},
                      "curve": curve, "knee_tokens_at_90pct": knee,
                      "paper_context": "the paper's reward-model forward saturates near 2048 batched tokens on an A100 "
                                       "(Section Lazy Verification); this curve is the attention call alone on a B200"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5", choices=sorted(WORKLOADS) + ["lv-sweep"],
                    help="lv-sweep: verification-attention throughput against the number of batched step tokens")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink the number of problems (debugging only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tiles-2cta", action="store_true",
                    help="run the tile items on the two-CTAs-per-SM kernel (64-key tiles) instead of the default one")
    ap.add_argument("--graph", action="store_true",
                    help="also time the step as a CUDA graph replay (reported as ms_per_step_cuda_graph)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-depth", type=int, default=3,
                    help="independent (host buffers, device arena, stream) sets the end-to-end leg alternates between")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the c2 / c3 / c4 and next-row measurements that the default run appends (`workloads`, `next_rows`)")
    ap.add_argument("--profiler-range", action="store_true",
                    help="bracket the timed region with cudaProfilerStart/Stop (for ncu --profile-from-start off)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    from paper_2609_39334_b200 import synth

    if args.workload == "lv-sweep":
        return lv_sweep(args)
    cfg_idx = WORKLOADS[args.workload]

    # ---------------------------------------------------------------------------------------------- reference arm
    if args.impl == "reference":
        if rank != 0:
            return
        import oracle
        oracle.build()
        dev = "cuda:0" if torch.cuda.is_available() else "cpu"
        w = synth.make_config(cfg_idx, device=dev, scale=args.scale)
        # every step is one pass over a bounded sample; the sample shrinks with the number of passes so that the whole
        # run stays within a few minutes (the default 10 + 1 passes: about a quarter of the single-pass sample each)
        passes = max(args.steps, 1) + min(args.warmup, 1)
        scale = min(1.0, 4.0 / passes)
        sample = oracle_sample(w, budget_scale=scale, min_paths=MIN_ORACLE_SAMPLE if scale >= 1.0 else 32)
        sub = synth.extract_subworkload(w, sample)
        del w
        if dev != "cpu":
            torch.cuda.empty_cache()
        sec = time_oracle(sub, max(args.steps, 1), min(args.warmup, 1))
        tokens = int(sub.path_q_len.astype(np.int64).sum())
        val = tokens / sec
        what = (f"{len(sample)} unique paths of {args.workload} ({int((sub.path_q_len > 1).sum())} verification, "
                f"{int((sub.path_q_len == 1).sum())} decode), {tokens} query tokens per step")
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": what},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.host_cores(), "kind": "oracle", "sample": what},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return

    # ---------------------------------------------------------------------------------------------------- our arm
    assert torch.cuda.is_available(), "bench.py needs a GPU (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2609_39334_b200 import binding as B
    from paper_2609_39334_b200.pipeline import DevicePipeline
    B.lib()

    # every rank its own problems: same shapes, different seed
    from paper_2609_39334_b200 import replicas
    w = replicas.replica_workload(synth.make_config, cfg_idx, rank, device=dev, scale=args.scale, poison=True)
    pipe = DevicePipeline(w, dev, attn_flags=B.SS_FLAG_TILES_2CTA if args.tiles_2cta else 0)
    kv_bytes = pipe.kv_pool.numel() * 2
    flush = None
    if kv_bytes < 4 * L2_BYTES:
        flush = L2Flush(dev)

    def sync_all():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize(dev)

    # warm-up (also the functional check of the device status)
    for _ in range(max(args.warmup, 1) if args.warmup else 0):
        pipe.step()
    torch.cuda.synchronize(dev)
    if args.warmup:
        st = B.ss_last_device_status(pipe.attn_ws)
        if st != B.SS_OK:
            raise B.SpecScaleError(st, "warm-up")

    clocks = ClockSampler(local_rank)
    if rank == 0:
        clocks.start()
        time.sleep(0.15)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    B.ss_profile_read()
    B.ss_profile_enable(True)
    launches0 = B.ss_launch_count()
    sync_all()
    if args.profiler_range:
        torch.cuda.profiler.start()
    for i in range(args.steps):
        if flush is not None:
            flush.fill_(i & 0xff)       # evicts the pool from L2 between iterations (outside the timed events)
        ev[i][0].record()
        pipe.step()
        ev[i][1].record()
    sync_all()
    if args.profiler_range:
        torch.cuda.profiler.stop()
    launches = B.ss_launch_count() - launches0
    B.ss_profile_enable(False)
    phase_ms, phase_calls = B.ss_profile_read()
    # the same K steps once more without the per-phase events of the library's profiler (they cost a few microseconds
    # per phase and keep consecutive kernels from overlapping their launch latency): reported beside the main number
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    sync_all()
    for i in range(args.steps):
        if flush is not None:
            flush.fill_(i & 0xff)
        ev2[i][0].record()
        pipe.step()
        ev2[i][1].record()
    sync_all()
    # optionally once more as a CUDA graph replay (one graph = one whole step): what a serving loop that calls the same
    # step shape repeatedly would pay; every call of the library is stream-ordered and allocation-free, so it captures
    graph_ms = None
    if args.graph:
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            pipe.step()                                   # first-use initialisation outside the capture
        torch.cuda.current_stream(dev).wait_stream(side)
        sync_all()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            pipe.step()
        ev3 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        sync_all()
        for i in range(args.steps):
            if flush is not None:
                flush.fill_(i & 0xff)
            ev3[i][0].record()
            g.replay()
            ev3[i][1].record()
        sync_all()
        graph_ms = replicas.max_over_ranks(float(sum(a.elapsed_time(b) for a, b in ev3)), dev) / args.steps
    clk = clocks.stop() if rank == 0 else None
    plain_ms = replicas.max_over_ranks(float(sum(a.elapsed_time(b) for a, b in ev2)), dev) / args.steps
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = replicas.max_over_ranks(float(sum(step_ms)), dev)
    ms_per_step = total_ms / args.steps
    st = B.ss_last_device_status(pipe.attn_ws)
    if st != B.SS_OK:
        raise B.SpecScaleError(st, "timed region")

    U = int(pipe.num_unique.item())
    unique_paths = pipe.unique_paths[:U].cpu().numpy()
    work = algorithmic_work(w, unique_paths)
    tokens = work["tokens"]
    value = replicas.whole_job_rate(tokens, ms_per_step)

    # ---- roofline of the attention kernels (per launch, CUDA events on the launching stream) -----------------
    peaks = load_peaks()
    long_step = total_ms > 1000.0
    tensor_peak = peaks["bf16_sustained"] if long_step else peaks["bf16_burst"]
    traffic = {}
    tpath = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if os.path.exists(tpath) and args.scale == 1.0:
        with open(tpath) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 3 and parts[0] == args.workload:
                    traffic[parts[1]] = float(parts[2])
    roofs = {}
    if phase_calls["tiles"]:
        t_ms = phase_ms["tiles"] / phase_calls["tiles"]
        ach = work["tile_flops"] / (t_ms * 1e-3) / 1e12
        roofs["tiles"] = {"kernel": "tile_items_umma_kernel" if args.tiles_2cta else "tile_items_umma_split_kernel",
                          "bound": "tensor", "achieved": ach, "peak": tensor_peak,
                          "unit": "TFLOP/s", "frac": ach / tensor_peak, "traffic": traffic.get("tiles"),
                          "ms_per_launch": t_ms, "peak_kind": f"{peaks['source']} {'sustained' if long_step else 'burst'}",
                          "frac_of_nominal": ach / NOMINAL_BF16_TFLOPS, "nominal_peak": NOMINAL_BF16_TFLOPS,
                          "frac_of_sustained": ach / peaks["bf16_sustained"],
                          "ctas_per_sm": 2 if args.tiles_2cta else 1}
    if phase_calls["leaves"]:
        t_ms = phase_ms["leaves"] / phase_calls["leaves"]
        ach = work["leaf_bytes"] / (t_ms * 1e-3) / 1e9
        roofs["leaves"] = {"kernel": "leaf_items_kernel", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                           "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": traffic.get("leaves"),
                           "ms_per_launch": t_ms, "peak_kind": f"{peaks['source']} copy",
                           "frac_of_nominal": ach / NOMINAL_HBM_GBS, "nominal_peak": NOMINAL_HBM_GBS}
    dominant = max(roofs, key=lambda k: roofs[k]["ms_per_launch"]) if roofs else None
    attn_ms = sum(phase_ms.values()) / max(phase_calls["plan"], 1)

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "paths": w.num_paths, "unique_paths": U, "query_tokens": tokens,
                   "heads": f"{w.num_q_heads}q/{w.num_kv_heads}kv", "kv_pool_gb": kv_bytes / 1e9,
                   "l2": "inputs larger than L2" if flush is None else L2Flush.NOTE,
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU"},
        "gpu_launches": int(launches),
        "attention_ms_per_step": attn_ms,
        "attention_tokens_per_s": world * tokens / (attn_ms * 1e-3) if attn_ms > 0 else None,
        "ms_per_step_median": float(np.median(step_ms)), "ms_per_step_min": float(min(step_ms)),
        "ms_per_step_without_phase_events": plain_ms,
        "ms_per_step_cuda_graph": graph_ms,
        "phase_ms_per_step": {k: (phase_ms[k] / phase_calls[k] if phase_calls[k] else 0.0) for k in phase_ms},
        "roofline": roofs.get(dominant) if dominant else None,
        "roofline_phases": roofs,
        "unique_kv_gb": work["unique_kv_bytes"] / 1e9,
        "clocks": clk,
    }

    # ---- end to end: ss_candidate_step_host - inputs from pinned host memory, results back to the host, every step --
    if not args.no_e2e:
        from paper_2609_39334_b200.pipeline import HostStepPipeline
        host = HostStepPipeline(pipe, depth=args.e2e_depth, compact=True)
        slim = host.measure_traffic()                     # (bytes per step as the call really moves them)
        for i in range(args.e2e_depth):
            host.submit(i)
        host.synchronize()
        host.results(0)                                   # raises on a device-side error
        sync_all()
        n_e2e = max(2 * args.steps, 2 * args.e2e_depth)   # (twice K: the first and the last step copy one way only)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream(dev)
        e0.record(cur)
        for s_ in host.sets:
            s_["stream"].wait_event(e0)
        for i in range(n_e2e):
            host.submit(i)
        for s_ in host.sets:
            cur.wait_stream(s_["stream"])
        e1.record(cur)
        sync_all()
        host.results(0)
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1) / n_e2e, dev)
        out["e2e"] = {"value": world * tokens / (e2e_ms * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": int(host.h2d_bytes), "d2h_bytes_per_step": int(host.d2h_bytes),
                      "ms_per_step": e2e_ms, "steps": n_e2e, "sets_in_flight": args.e2e_depth,
                      "api": "ss_candidate_step_host",
                      "live_rows_only_back": bool(slim),
                      "note": "KV pool stays resident (it is the cache); every step copies candidates and scores from "
                              "pinned host memory, copies every candidate's query rows in and returns the live rows of out / lse "
                              "(a small kernel writes them into the mapped host buffers) and all other results; steps "
                              "alternate between independent (host buffers, device arena, stream) sets so copies "
                              "overlap kernels"}
        del host

    # ---- CPU oracle beside it (rank 0, N = 1 only) ----------------------------------------------------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        sample = oracle_sample(w)
        sub = synth.extract_subworkload(w, sample)
        sec = time_oracle(sub, 1, 0)
        stok = int(sub.path_q_len.astype(np.int64).sum())
        out["cpu_baseline"] = {
            "value": stok / sec, "unit": UNIT, "cores": oracle.host_cores(), "kind": "oracle",
            "sample": f"{len(sample)} unique paths of {args.workload} ({int((sub.path_q_len > 1).sum())} verification, "
                      f"{int((sub.path_q_len == 1).sum())} decode), {stok} query tokens, {sec:.1f} s"}

    # ---- the other benchmark configurations and the rows beyond the core path (default run, rank 0, N = 1) ------------
    if rank == 0 and world == 1 and args.workload == "c5" and args.scale == 1.0 and not args.no_workloads:
        del pipe
        w.kv_pool = None
        w.q = None
        torch.cuda.empty_cache()
        small_flush = L2Flush(dev)
        out["workloads"] = {name: small_workload(name, dev, small_flush, peaks) for name in ("c2", "c3", "c4")}
        out["next_rows"] = next_rows(dev, small_flush, peaks)
        curve, knee = lv_curve(dev, small_flush, 20, 3)
        out["next_rows"]["lv_sweep"] = {"curve": curve, "knee_tokens_at_90pct": knee,
                                        "paper_context": "reward-model forward saturates near 2048 batched tokens on an A100"}
        del small_flush

    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
