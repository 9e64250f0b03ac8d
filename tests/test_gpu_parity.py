"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Bars: dedup / remap / top-k bit-exact; attention |out - oracle| <= 2e-2 max and <= 2e-3 mean, |lse - oracle| <= 1e-3
(bf16 inputs ~N(0,1), fp64 oracle).  Tighter internal gates (see TIGHT below) catch indexing slips that those bars
would let through on long paths: dropping one 16-token page of a 4672-key path moves the output by only ~1.4e-3.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_39334_b200 import binding as B
from paper_2609_39334_b200 import synth
from paper_2609_39334_b200.pipeline import DevicePipeline

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

OUT_MAX, OUT_MEAN, LSE_MAX = 2e-2, 2e-3, 1e-3          # official
# Internal gates, set from the errors observed on a B200 (SS_PARITY_LOG collects them):
#   * paths of >= 256 keys (every benchmark configuration): observed out max <= 9.8e-4, mean <= 1.1e-4 -> 4e-3 / 3e-4;
#   * any length, element by element: |err| <= 2^-8 |exact| + 2.5e-3.  The bf16 rounding of the output is at most 2^-9
#     relative; rounding P to bf16 before P V perturbs every term p_j v_j by up to 2^-9 relative, which does not shrink
#     with |exact| when terms cancel: with a few dominant keys and |v| up to ~4 that is up to a few 1e-3 (observed:
#     1.4e-3 beyond the relative part on 100-key verification rows, 5.4e-3 in all on 5-key paths with outputs near 3);
#   * LSE: fp32 sums of ex2.approx values, observed <= 2.6e-6 -> 2e-5 (a causal mask that is off by one key moves the LSE
#     of a 4672-key row by 2e-4).
TIGHT_OUT_MAX, TIGHT_OUT_MEAN, TIGHT_LSE = 4e-3, 3e-4, 2e-5
TIGHT_REL, TIGHT_ABS = 2.0 ** -8, 2.5e-3
LONG_PATH = 256


def tight_gates(out, o_ref, lerr, min_len):
    err = np.abs(out - o_ref)
    assert (err <= TIGHT_REL * np.abs(o_ref) + TIGHT_ABS).all(), float((err - TIGHT_REL * np.abs(o_ref)).max())
    assert lerr <= TIGHT_LSE, lerr
    if min_len >= LONG_PATH:
        assert err.max() <= TIGHT_OUT_MAX and err.mean() <= TIGHT_OUT_MEAN, (err.max(), err.mean())


def log_observed(name, out_max, out_mean, lse_max):
    """Appends the observed errors of one comparison to the file named by SS_PARITY_LOG (if set), so that the gates
    below can be set from measurements."""
    path = os.environ.get("SS_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(f"{name} out_max={out_max:.3e} out_mean={out_mean:.3e} lse_max={lse_max:.3e}\n")


def check_dedup(r, w):
    ref = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
    assert r["num_unique"] == ref["num_unique"]
    for key in ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out"):
        assert np.array_equal(r[key], ref[key]), key
    return ref


def check_topk(r, w):
    s_ref, k_ref = oracle.topk(w.scores, w.seg_offsets, w.top_k)
    assert np.array_equal(r["survivors"], s_ref)
    assert np.array_equal(r["keep"], k_ref)


def sample_unique(ref, w, max_paths, seed=0):
    """Indices INTO the unique list: all if few, else a seeded sample that contains the extremes."""
    U = ref["num_unique"]
    if U <= max_paths:
        return np.arange(U)
    uniq = ref["unique_paths"]
    lens = np.asarray([w.node_kv_len[w.path_leaf_node[u]] for u in uniq])
    T = w.path_q_len[uniq]
    must = {0, U - 1, int(lens.argmin()), int(lens.argmax()), int(T.argmax()), int(T.argmin())}
    mult = ref["multiplicity"]
    if (mult > 1).any():
        must.add(int(np.nonzero(mult > 1)[0][0]))
    rng = np.random.default_rng(seed)
    rest = rng.choice(U, size=max_paths - len(must), replace=False)
    return np.asarray(sorted(must | set(int(x) for x in rest)))[:max_paths]


def check_attention(r, w, ref, max_paths=48, tight=True, host_w=None):
    """Compares the GPU rows of a sample of unique paths with the oracle."""
    sel = sample_unique(ref, w, max_paths)
    uniq = ref["unique_paths"][sel]
    src = host_w if host_w is not None else w
    o_ref, l_ref = oracle.tree_attention_workload(src, paths=uniq)
    # rows of the selected unique paths in the compacted GPU output
    T_u = w.path_q_len[ref["unique_paths"]].astype(np.int64)
    off = np.concatenate([[0], np.cumsum(T_u)])
    rows = np.concatenate([np.arange(off[i], off[i + 1]) for i in sel])
    out, lse = r["out"][rows], r["lse"][rows]
    assert np.isfinite(out).all(), "NaN/inf in attention output (poisoned slot read?)"
    err = np.abs(out - o_ref)
    fin = np.isfinite(l_ref)
    assert np.array_equal(np.isfinite(lse), fin)
    lerr = np.abs(lse[fin] - l_ref[fin]).max() if fin.any() else 0.0
    log_observed(f"{w.name} tight={tight}", err.max(), err.mean(), lerr)
    assert err.max() <= OUT_MAX and err.mean() <= OUT_MEAN and lerr <= LSE_MAX, (err.max(), err.mean(), lerr)
    if tight:
        tight_gates(out, o_ref, lerr, min(src.path_kv_len(int(u)) for u in uniq))
    return err.max(), err.mean(), lerr


MODES = [("fast", 0), ("two_cta", B.SS_FLAG_TILES_2CTA), ("no_tcgen05", B.SS_FLAG_NO_TCGEN05),
         ("generic", B.SS_FLAG_FORCE_GENERIC)]


# =========================================================================================================
# whole pipeline on the benchmark configurations
# =========================================================================================================
@pytest.mark.parametrize("mode,flags", MODES)
@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_pipeline_configs(cfg, mode, flags):
    if mode == "generic" and cfg in (3,):
        scale = 0.25
    else:
        scale = 1.0
    w = synth.make_config(cfg, scale=scale)
    pipe = DevicePipeline(w, DEV, attn_flags=flags | B.SS_FLAG_VALIDATE)
    pipe.step()
    r = pipe.results()
    ref = check_dedup(r, w)
    check_topk(r, w)
    check_attention(r, w, ref, max_paths=40 if cfg != 3 else 12)
    # duplicates read their result through path_to_unique: identical by construction
    assert r["num_unique"] <= w.num_paths


def test_pipeline_config1_all_rows_and_fullseq_dedup():
    w = synth.make_config(1)
    pipe = DevicePipeline(w, DEV)
    pipe.step()
    r = pipe.results()
    ref = check_dedup(r, w)
    check_attention(r, w, ref, max_paths=8)
    # config 1 also de-duplicates on the full prefix+suffix token sequence with a null context
    rng = np.random.default_rng(1)
    prefix = rng.integers(0, synth.VOCAB, size=256).astype(np.int32)
    seqs = [np.concatenate([prefix, w.tok_ids[w.tok_offsets[i]:w.tok_offsets[i + 1]]]) for i in range(8)]
    ids = np.concatenate(seqs).astype(np.int32)
    off = np.concatenate([[0], np.cumsum([len(s) for s in seqs])]).astype(np.int64)
    got = run_dedup(ids, off, None, None)
    want = oracle.dedup(ids, off)
    for key in ("canon", "path_to_unique", "unique_paths", "multiplicity"):
        assert np.array_equal(got[key], want[key])


# =========================================================================================================
# dedup
# =========================================================================================================
def run_dedup(ids, off, ctx, slot, flags=0):
    n = len(off) - 1
    dev = torch.device(DEV)
    t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(dev)
    ids_t = t(ids if len(ids) else np.zeros(1, np.int32), np.int32)
    i32 = dict(dtype=torch.int32, device=dev)
    m = max(n, 1)
    canon, p2u, uniq, mult = (torch.full((m,), -7, **i32) for _ in range(4))
    slot_out = torch.full((m,), -7, **i32) if slot is not None else None
    nu = torch.full((1,), -7, **i32)
    ws = B.alloc_workspace(B.ss_dedup_workspace_bytes(n), dev)
    B.ss_dedup_paths(ids_t, t(off, np.int64), t(ctx, np.int64), t(slot, np.int32), n, flags, canon, p2u, uniq, mult,
                     slot_out, nu, ws)
    torch.cuda.synchronize()
    U = int(nu.item())
    return dict(num_unique=U, canon=canon[:n].cpu().numpy(), path_to_unique=p2u[:n].cpu().numpy(),
                unique_paths=uniq[:U].cpu().numpy(), multiplicity=mult[:U].cpu().numpy(),
                slot_out=None if slot is None else slot_out[:n].cpu().numpy())


def dedup_case(rng, n, alphabet, max_len, n_ctx):
    lens = rng.integers(0, max_len + 1, size=n)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    ids = rng.integers(0, alphabet, size=int(off[-1])).astype(np.int32)
    ctx = rng.integers(0, n_ctx, size=n).astype(np.int64)
    slot = rng.integers(0, 1 << 20, size=n).astype(np.int32)
    return ids, off, ctx, slot


@pytest.mark.parametrize("flags", [0, B.SS_FLAG_WEAK_HASH])
@pytest.mark.parametrize("n,alphabet,max_len,n_ctx", [
    (1, 3, 4, 1), (2, 2, 2, 1), (37, 2, 3, 2), (300, 3, 5, 2), (1025, 3, 5, 2), (2049, 4, 6, 3), (4096, 3, 5, 2), (4097, 3, 5, 2), (5000, 2, 40, 1), (8192, 3, 6, 2), (12000, 4, 6, 3),
    (16384, 3, 5, 2), (16385, 3, 5, 2), (20000, 50, 3, 4),
])
def test_dedup_random_collision_heavy(n, alphabet, max_len, n_ctx, flags):
    rng = np.random.default_rng(n * 31 + alphabet)
    ids, off, ctx, slot = dedup_case(rng, n, alphabet, max_len, n_ctx)
    got = run_dedup(ids, off, ctx, slot, flags)
    want = oracle.dedup(ids, off, ctx, slot)
    assert got["num_unique"] == want["num_unique"]
    for key in ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out"):
        assert np.array_equal(got[key], want[key]), key


def test_dedup_edge_cases():
    got = run_dedup(np.zeros(0, np.int32), np.zeros(1, np.int64), None, None)
    assert got["num_unique"] == 0
    # all empty sequences, null ctx: one class
    got = run_dedup(np.zeros(0, np.int32), np.zeros(6, np.int64), None, None)
    assert got["num_unique"] == 1 and list(got["canon"]) == [0] * 5 and list(got["multiplicity"]) == [5]
    # all identical long sequences
    seq = np.arange(1000, dtype=np.int32)
    ids = np.tile(seq, 64)
    off = (np.arange(65) * 1000).astype(np.int64)
    got = run_dedup(ids, off, None, np.arange(64, dtype=np.int32))
    assert got["num_unique"] == 1 and list(got["slot_out"]) == [0] * 64
    # differ only in the last token / only in length / only in ctx
    ids = np.asarray([1, 2, 3, 1, 2, 4, 1, 2, 1, 2, 3], np.int32)
    off = np.asarray([0, 3, 6, 8, 11], np.int64)
    got = run_dedup(ids, off, np.asarray([0, 0, 0, 1], np.int64), None)
    assert list(got["canon"]) == [0, 1, 2, 3]
    got = run_dedup(ids, off, np.asarray([5, 5, 5, 5], np.int64), None)
    assert list(got["canon"]) == [0, 1, 2, 0]
    # tok_offsets that do not start at zero
    got = run_dedup(np.asarray([9, 9, 7, 7, 7, 7], np.int32), np.asarray([2, 4, 6], np.int64), None, None)
    assert list(got["canon"]) == [0, 0]


def test_dedup_paper_example_on_gpu():
    got = run_dedup(np.asarray([1055, 1055, 1055, 429], np.int32), np.arange(5, dtype=np.int64), np.zeros(4, np.int64), None)
    assert list(got["multiplicity"]) == [3, 1]


def test_dedup_idempotent_and_permutation_invariant_on_gpu():
    rng = np.random.default_rng(77)
    ids, off, ctx, slot = dedup_case(rng, 4000, 3, 4, 2)
    r = run_dedup(ids, off, ctx, None)
    seqs = [ids[off[i]:off[i + 1]] for i in range(4000)]
    u = r["unique_paths"]
    ids2 = np.concatenate([seqs[i] for i in u]).astype(np.int32)
    off2 = np.concatenate([[0], np.cumsum([len(seqs[i]) for i in u])]).astype(np.int64)
    r2 = run_dedup(ids2, off2, ctx[u], None)
    assert r2["num_unique"] == len(u) and np.array_equal(r2["canon"], np.arange(len(u)))
    perm = rng.permutation(4000)
    ids3 = np.concatenate([seqs[i] for i in perm]).astype(np.int32) if len(ids) else ids
    off3 = np.concatenate([[0], np.cumsum([len(seqs[i]) for i in perm])]).astype(np.int64)
    r3 = run_dedup(ids3, off3, ctx[perm], None)
    assert r3["num_unique"] == r["num_unique"]
    inv = np.argsort(perm)
    cls_min = {}
    for i in range(4000):
        c = int(r["canon"][i])
        cls_min[c] = min(cls_min.get(c, 1 << 30), int(inv[i]))
    assert all(int(r3["canon"][inv[i]]) == cls_min[int(r["canon"][i])] for i in range(4000))


# =========================================================================================================
# top-k
# =========================================================================================================
def run_topk(scores, seg, k):
    dev = torch.device(DEV)
    n, P = len(scores), len(seg) - 1
    sc = torch.from_numpy(np.ascontiguousarray(scores if n else np.zeros(1, np.float32), dtype=np.float32)).to(dev)
    sg = torch.from_numpy(np.ascontiguousarray(seg, dtype=np.int32)).to(dev)
    surv = torch.full((max(P, 1), k), -9, dtype=torch.int32, device=dev)
    keep = torch.full((max(n, 1),), 7, dtype=torch.uint8, device=dev)
    ws = B.alloc_workspace(B.ss_topk_workspace_bytes(n), dev)
    B.ss_topk_prune(sc, sg, P, n, k, surv, keep, ws)
    torch.cuda.synchronize()
    return surv[:P].cpu().numpy(), keep[:n].cpu().numpy()


@pytest.mark.parametrize("sizes,k", [
    ([32] * 8, 8), ([0, 5, 0, 1, 70], 4), ([4096], 64), ([5000, 3, 9000], 100), ([20000], 1), ([7], 16), ([256] * 64, 64),
])
def test_topk_vs_oracle(sizes, k):
    rng = np.random.default_rng(sum(sizes) + k)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    n = int(seg[-1])
    for variant in range(2):
        if variant == 0:
            sc = rng.random(n).astype(np.float32)
        else:                                   # tie-heavy, large mass at the perfect score
            sc = (rng.integers(0, 9, size=n) / 8.0).astype(np.float32)
            sc[rng.random(n) < 0.3] = 1.0
        surv, keep = run_topk(sc, seg, k)
        s_ref, k_ref = oracle.topk(sc, seg, k)
        assert np.array_equal(surv, s_ref) and np.array_equal(keep, k_ref)


def test_topk_special_values_and_gaps():
    sc = np.asarray([0.0, -0.0, np.nan, 0.5, np.nan, -1.0, np.inf, -np.inf, 3.0, 3.0], np.float32)
    surv, keep = run_topk(sc, [0, 8], 8)          # candidates 8, 9 belong to no segment
    assert list(surv[0]) == [6, 3, 0, 1, 5, 7, 2, 4] and list(keep[8:]) == [0, 0]
    s_ref, k_ref = oracle.topk(sc, [0, 8], 3)
    surv, keep = run_topk(sc, [0, 8], 3)
    assert np.array_equal(surv, s_ref) and np.array_equal(keep[:8], k_ref[:8])


def test_topk_beam_bookkeeping_on_gpu():
    rng = np.random.default_rng(3)
    for N, M in [(4, 4), (8, 4), (16, 4), (32, 4)]:
        sc = rng.random(N).astype(np.float32)
        surv, keep = run_topk(sc, [0, N], N // M)
        assert int(keep.sum()) == N // M and set(surv[0]) == set(np.argsort(-sc, kind="stable")[:N // M])


# =========================================================================================================
# attention: shapes beyond the configs, closed forms, invariances
# =========================================================================================================
def attention_only(w, flags=0, sm_scale=0.0):
    pipe = DevicePipeline(w, DEV, attn_flags=flags | B.SS_FLAG_VALIDATE, sm_scale=sm_scale)
    pipe.dedup()
    pipe.compact_unique()
    pipe.attention()
    r = pipe.results()
    ref = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
    return r, ref


SHAPES = [
    # name, Hq, Hkv, levels, fanout, problems, leaf range, T-fn, dup
    ("gqa1_deep", 4, 4, [64, 32, 16], [2, 3, 2], 2, (0, 70), lambda i, n, rng: 1, 0.2),
    ("gqa7_mixed", 28, 4, [192], [9], 3, (0, 150), lambda i, n, rng: 1 if i % 3 else int(rng.integers(2, 50)), 0.1),
    ("gqa8_verify_ragged", 16, 2, [128, 64], [2, 5], 2, (1, 200), lambda i, n, rng: int(rng.integers(16, 129)), 0.0),
    ("gqa16_decode", 32, 2, [256], [40], 2, (0, 300), lambda i, n, rng: 1, 0.3),
    ("gqa2_small_T", 8, 4, [48], [6], 2, (3, 40), lambda i, n, rng: int(rng.integers(1, 6)), 0.0),
    ("gqa32_generic_decode", 32, 1, [64], [5], 1, (1, 90), lambda i, n, rng: 1 + (i % 2) * 20, 0.0),
    ("no_prefix", 12, 2, [0], [7], 2, (0, 130), lambda i, n, rng: 1 + (i % 2) * 17, 0.0),
    ("long_prefix_few_paths", 8, 2, [4096], [3], 1, (5, 600), lambda i, n, rng: 1, 0.0),
]


@pytest.mark.parametrize("mode,flags", MODES)
@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_attention_shapes(shape, mode, flags):
    name, Hq, Hkv, levels, fanout, problems, leaf, qfn, dup = shape
    w = synth.build_tree_workload(name, 1234, Hq, Hkv, levels, fanout, problems, leaf, qfn, dup_frac=dup)
    r, ref = attention_only(w, flags)
    check_attention(r, w, ref, max_paths=64)


@pytest.mark.parametrize("seed", range(8))
def test_attention_random_trees(seed):
    """Seeded random tree shapes (depth, fan-out, head grouping, leaf and step lengths, duplicates) through the
    default kernels: item boundaries, ragged tiles, page tails and empty leaves fall differently in each."""
    rng = np.random.default_rng(9000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 6, 7, 8, 16]))
    depth = int(rng.integers(1, 4))
    levels = [int(rng.choice([0, 16, 40, 128, 300, 700])) for _ in range(depth)]
    fanout = [int(rng.integers(1, 6)) for _ in range(depth - 1)] + [int(rng.integers(2, 40))]
    leaf = (int(rng.integers(0, 3)), int(rng.choice([20, 130, 400])))
    style = int(rng.integers(0, 3))

    def qfn(i, n, r):
        if style == 0:
            return 1
        if style == 1:
            return int(r.integers(1, 140))
        return 1 if i % 2 else int(r.integers(16, 129))

    w = synth.build_tree_workload(f"fuzz{seed}", 77000 + seed, Hkv * G, Hkv, levels, fanout, int(rng.integers(1, 4)), leaf, qfn,
                                  dup_frac=float(rng.choice([0.0, 0.2])))
    r, ref = attention_only(w, 0)
    check_attention(r, w, ref, max_paths=48)


@pytest.mark.parametrize("mode,flags", MODES)
def test_attention_closed_forms(mode, flags):
    """Q == 0 => lse = ln(visible), out = mean of the visible V rows; with V[j,:] = position j (< 256, exact in
    bf16) that mean is (visible-1)/2.  Catches off-by-one in masks, page order and node lengths at tight
    tolerance."""
    for levels, fanout, T in [([64], [5], 1), ([32, 48], [2, 3], 1), ([80], [3], 24), ([64], [2], 3)]:
        w = synth.build_tree_workload("cf", 99, 8, 2, levels, fanout, 1, (0, 100), lambda i, n, rng: T)
        w.q.zero_()
        for p in range(w.num_paths):
            pos = 0
            for n in w.chain(int(w.path_leaf_node[p])):
                pages = w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]]
                for j in range(int(w.node_kv_len[n])):
                    w.kv_pool[int(pages[j // 16]), 1, :, j % 16, :] = float(pos)
                    pos += 1
            assert pos <= 256
        r, ref = attention_only(w, flags)
        row = 0
        for u in ref["unique_paths"]:
            L = w.path_kv_len(int(u))
            for t in range(T):
                vis = L - T + t + 1
                if vis <= 0:
                    assert np.all(r["out"][row] == 0) and np.all(np.isneginf(r["lse"][row]))
                else:
                    np.testing.assert_allclose(r["lse"][row], math.log(vis), atol=2e-5)
                    # bf16 output rounding: relative 2^-9
                    np.testing.assert_allclose(r["out"][row], (vis - 1) / 2.0, rtol=2.0 ** -8, atol=1e-6)
                row += 1


def test_attention_page_permutation_and_explicit_scale():
    w = synth.build_tree_workload("perm", 5, 12, 2, [128], [6], 2, (1, 120), lambda i, n, rng: 1 + (i % 2) * 30)
    r1, ref = attention_only(w, sm_scale=0.05)
    o_ref, l_ref = oracle.tree_attention_workload(w, paths=ref["unique_paths"], sm_scale=0.05)
    tight_gates(r1["out"], o_ref, np.abs(r1["lse"] - l_ref).max(), 0)
    rng = np.random.default_rng(0)
    perm = rng.permutation(w.num_pages)
    new_pool = torch.empty_like(w.kv_pool)
    new_pool[torch.from_numpy(perm)] = w.kv_pool
    w.kv_pool = new_pool
    w.node_pages = perm[w.node_pages].astype(np.int32)
    r2, _ = attention_only(w, sm_scale=0.05)
    # only the physical page ids differ: every item sees the same numbers in the same order
    assert np.array_equal(r2["out"], r1["out"]) and np.array_equal(r2["lse"], r1["lse"])


def test_attention_on_a_limited_number_of_sms_gives_the_same_result():
    """`max_sms` only changes how many blocks the tile and leaf kernels launch (the host-buffer step keeps a few SMs for
    its copy kernel): every item is computed by one block in the same order of operations, so the result is the same
    to the bit, and a value above the device's SM count means all of them."""
    w = synth.build_tree_workload("sms", 31, 12, 2, [256], [9], 3, (1, 600), lambda i, n, rng: 1 + (i % 3 == 0) * 40)
    outs = []
    for sms in (0, 3, 1, 100000):
        pipe = DevicePipeline(w, DEV, attn_flags=B.SS_FLAG_VALIDATE)
        pipe.desc.max_sms = sms
        pipe.dedup()
        pipe.compact_unique()
        pipe.attention()
        outs.append(pipe.results())
    ref = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
    check_attention(outs[0], w, ref, max_paths=16)
    for r in outs[1:]:
        assert np.array_equal(r["out"], outs[0]["out"]) and np.array_equal(r["lse"], outs[0]["lse"])


def test_attention_flat_per_path_page_tables():
    """A cache that keeps one flat page list per sequence is the tree form with one node per path: a root that is its
    own leaf, whose page list is the whole sequence.  Same pool, same queries: the results must agree with the oracle
    on the flat description and (within the gates) with the shared-prefix description of the same data."""
    import copy
    w = synth.build_tree_workload("flat", 21, 8, 2, [64], [5], 2, (3, 150), lambda i, n, rng: 1 + (i % 2) * 23)
    r_tree, ref = attention_only(w)
    flat = copy.copy(w)
    parents, lens, pages, offs = [], [], [], [0]
    for p in range(w.num_paths):
        chain, n = [], int(w.path_leaf_node[p])
        while n >= 0:
            chain.append(n)
            n = int(w.node_parent[n])
        pl, total = [], 0
        for n in reversed(chain):                              # inner nodes hold whole pages, so the lists concatenate
            pl += list(w.node_pages[w.node_page_offsets[n]:w.node_page_offsets[n + 1]])
            total += int(w.node_kv_len[n])
        parents.append(-1)
        lens.append(total)
        pages += pl
        offs.append(len(pages))
    flat.node_parent = np.asarray(parents, np.int32)
    flat.node_kv_len = np.asarray(lens, np.int32)
    flat.node_pages = np.asarray(pages, np.int32)
    flat.node_page_offsets = np.asarray(offs, np.int64)
    flat.path_leaf_node = np.arange(w.num_paths, dtype=np.int32)
    flat.slot_in = flat.path_leaf_node.copy()
    r_flat, ref_flat = attention_only(flat)
    assert np.array_equal(ref_flat["unique_paths"], ref["unique_paths"])
    o_ref, l_ref = oracle.tree_attention_workload(flat, paths=ref_flat["unique_paths"])
    tight_gates(r_flat["out"], o_ref, np.abs(r_flat["lse"] - l_ref).max(), 0)
    assert np.abs(r_flat["out"] - r_tree["out"]).max() <= 2 * TIGHT_ABS + TIGHT_REL * np.abs(o_ref).max()


def test_attention_empty_and_degenerate():
    # every path empty: out = 0, lse = -inf
    w = synth.build_tree_workload("empty", 3, 4, 2, [0], [3], 1, (0, 0), lambda i, n, rng: 1)
    r, ref = attention_only(w)
    assert np.all(r["out"] == 0) and np.all(np.isneginf(r["lse"]))
    # no paths at all
    w = synth.build_tree_workload("p0", 3, 4, 2, [16], [0], 1, (0, 0), lambda i, n, rng: 1)
    pipe = DevicePipeline(w, DEV)
    pipe.step()
    assert pipe.results()["num_unique"] == 0


def test_attention_device_errors_are_reported():
    w = synth.build_tree_workload("bad", 3, 4, 2, [32], [3], 1, (1, 20), lambda i, n, rng: 1)
    pipe = DevicePipeline(w, DEV, attn_flags=B.SS_FLAG_VALIDATE)
    pipe.dedup()
    pipe.compact_unique()
    pipe.node_pages[0] = 10 ** 6                     # out-of-range page id: caught by the validator, never read
    pipe.attention()
    torch.cuda.synchronize()
    assert B.ss_last_device_status(pipe.attn_ws) == B.SS_ERR_BAD_INPUT
    pipe.node_pages[0] = int(w.node_pages[0])
    pipe.attention()
    torch.cuda.synchronize()
    assert B.ss_last_device_status(pipe.attn_ws) == B.SS_OK
    # a tree deeper than SS_MAX_DEPTH is refused, not walked
    deep = synth.build_tree_workload("deep", 3, 4, 2, [16] * 17, [1] * 17, 1, (1, 5), lambda i, n, rng: 1)
    pipe = DevicePipeline.__new__(DevicePipeline)
    with pytest.raises(B.SpecScaleError):
        DevicePipeline.__init__(pipe, deep, DEV)     # max_depth hint 18 > SS_MAX_DEPTH: rejected on the host


# =========================================================================================================
# full-size configuration 5 (the benchmark's workload, generated on the GPU): sampled outputs against the oracle
# =========================================================================================================
def test_config5_full_size_sampled_outputs():
    w = synth.make_config(5, device=DEV)                    # 16384 paths, ~42 GB pool, both modes, 20 % duplicates
    pipe = DevicePipeline(w, DEV)
    pipe.step()
    r = pipe.results()
    ref = check_dedup(r, w)                                 # dedup / remap bit-exact on all 16384 paths
    check_topk(r, w)
    U = ref["num_unique"]
    assert U < w.num_paths
    uniq = ref["unique_paths"]
    T = w.path_q_len[uniq]
    lens = w.node_kv_len[w.path_leaf_node[uniq]]
    rng = np.random.default_rng(5)
    ver, dec = np.nonzero(T > 1)[0], np.nonzero(T == 1)[0]
    # >= 128 unique paths: 44 verification paths (64 query tokens each) and 100 decode paths, plus the strata below
    pick = set(int(x) for x in rng.choice(ver, 44, replace=False)) | set(int(x) for x in rng.choice(dec, 100, replace=False))
    pick |= {int(dec[lens[dec].argmin()]), int(dec[lens[dec].argmax()]), int(ver[lens[ver].argmin()]),
             int(ver[lens[ver].argmax()]), 0, U - 1}
    dup_u = np.nonzero(ref["multiplicity"] > 1)[0]
    pick |= {int(dup_u[0]), int(dup_u[-1])}
    sel = np.asarray(sorted(pick))
    assert len(sel) >= 128 and (T[sel] > 1).sum() >= 40 and (T[sel] == 1).sum() >= 80
    sub = synth.extract_subworkload(w, uniq[sel])           # the needed pages and query rows, copied to the host
    o_ref, l_ref = oracle.tree_attention_workload(sub)
    off = np.concatenate([[0], np.cumsum(T.astype(np.int64))])
    rows = np.concatenate([np.arange(off[i], off[i + 1]) for i in sel])
    out, lse = r["out"][rows], r["lse"][rows]
    assert np.isfinite(out).all()
    err = np.abs(out - o_ref)
    lerr = np.abs(lse - l_ref).max()
    log_observed("config5_full", err.max(), err.mean(), lerr)
    assert err.max() <= OUT_MAX and err.mean() <= OUT_MEAN and lerr <= LSE_MAX, (err.max(), err.mean(), lerr)
    tight_gates(out, o_ref, lerr, LONG_PATH)


def test_attention_without_query_indirection_matches():
    """q_src_offsets = NULL (queries already compacted at q_offsets) gives the same result as reading them in place."""
    w = synth.build_tree_workload("noind", 77, 12, 2, [128], [6], 2, (1, 120), lambda i, n, rng: 1 + (i % 2) * 30,
                                  dup_frac=0.25)
    pipe = DevicePipeline(w, DEV)
    pipe.dedup()
    pipe.compact_unique()
    pipe.attention()
    r = pipe.results()
    U, tq = r["num_unique"], r["total_q"]
    src = pipe.u_q_src[:U].cpu().numpy()
    T = pipe.u_q_len[:U].cpu().numpy()
    rows = np.concatenate([np.arange(s, s + t) for s, t in zip(src, T)])
    q_compact = pipe.q[torch.from_numpy(rows).to(DEV)].contiguous()
    out = torch.empty_like(q_compact)
    lse = torch.empty((tq, w.num_q_heads), dtype=torch.float32, device=DEV)
    desc = B.make_attn_desc(
        num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads, kv_pool=pipe.kv_pool, node_parent=pipe.node_parent,
        node_kv_len=pipe.node_kv_len, node_page_offsets=pipe.node_page_offsets, node_pages=pipe.node_pages,
        total_node_pages=int(w.node_page_offsets[-1]), path_leaf_node=pipe.u_leaf[:U].contiguous(),
        path_q_len=pipe.u_q_len[:U].contiguous(), q_offsets=pipe.u_q_offsets[:U + 1].contiguous(), total_q=tq,
        q=q_compact, out=out, lse=lse)
    ws = B.alloc_workspace(B.ss_tree_attention_workspace_bytes(desc), DEV)
    B.ss_tree_attention(desc, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_OK
    assert np.array_equal(out.to(torch.float64).cpu().numpy(), r["out"])
    assert np.array_equal(lse.to(torch.float64).cpu().numpy(), r["lse"])


def test_attention_reports_too_small_workspace_from_the_device():
    """Sizing hints that are too low are caught by the planner (status read back), nothing is written out of bounds."""
    w = synth.build_tree_workload("hint", 9, 8, 2, [64], [12], 2, (1, 300), lambda i, n, rng: 1)
    pipe = DevicePipeline(w, DEV)
    pipe.dedup()
    pipe.compact_unique()
    good = B.ss_tree_attention_workspace_bytes(pipe.desc)
    pipe.desc.max_decode_paths = 3                       # 24 decode paths exist
    small = B.ss_tree_attention_workspace_bytes(pipe.desc)
    assert small < good
    canary = torch.full((4096,), 0x5A, dtype=torch.uint8, device=DEV)
    ws_all = torch.cat([B.alloc_workspace(small, DEV)[:small + (-small) % 256], canary])
    ws = ws_all[:ws_all.numel() - 4096]
    B.ss_tree_attention(pipe.desc, ws)
    torch.cuda.synchronize()
    assert B.ss_last_device_status(ws) == B.SS_ERR_WORKSPACE_TOO_SMALL
    assert bool((ws_all[-4096:] == 0x5A).all())         # nothing past the workspace was touched
    # host-side check: a workspace smaller than the query result is refused before any launch
    rc = B.ss_tree_attention(pipe.desc, ws[:1024], check=False)
    assert rc == B.SS_ERR_WORKSPACE_TOO_SMALL


# =========================================================================================================
# sizes at the edges of the supported range
# =========================================================================================================
EDGE_SHAPES = [
    # one very long path (decode and verification): many key tiles, one item per kv head
    ("long_decode", 8, 2, [16384], [1], 1, (2000, 2100), lambda i, n, rng: 1),
    ("long_verify", 8, 2, [8192], [2], 1, (100, 900), lambda i, n, rng: 128),
    # GQA group of 1 (128 tokens per tile) and of 128 (one token per tile), maximum step length
    ("gqa1_verify", 2, 2, [64], [3], 1, (0, 200), lambda i, n, rng: 128),
    ("gqa128_verify", 128, 1, [64], [2], 1, (0, 100), lambda i, n, rng: 5),
    # many tiny problems (more nodes than SMs), leaves that end exactly on page / tile boundaries
    ("many_problems", 12, 2, [32], [2], 300, (0, 20), lambda i, n, rng: 1 + (i % 2) * 15),
    ("exact_boundaries", 8, 2, [64], [4], 2, (64, 64), lambda i, n, rng: 1 + (i % 2) * 63),
    # depth at the limit: 15 shared levels + leaf
    ("depth16", 4, 2, [16] * 15, [1] * 14 + [3], 1, (1, 40), lambda i, n, rng: 1 + (i % 2) * 8),
]


@pytest.mark.parametrize("shape", EDGE_SHAPES, ids=[s[0] for s in EDGE_SHAPES])
def test_attention_edge_sizes(shape):
    name, Hq, Hkv, levels, fanout, problems, leaf, qfn = shape
    w = synth.build_tree_workload(name, 4321, Hq, Hkv, levels, fanout, problems, leaf, qfn)
    r, ref = attention_only(w)
    check_attention(r, w, ref, max_paths=24)


def test_dedup_large_batch():
    """One million candidate paths (far beyond the benchmark sizes): still bit-exact."""
    rng = np.random.default_rng(2024)
    n = 1_000_000
    ids, off, ctx, slot = dedup_case(rng, n, 30, 3, 8)
    got = run_dedup(ids, off, ctx, slot)
    want = oracle.dedup(ids, off, ctx, slot)
    assert got["num_unique"] == want["num_unique"]
    for key in ("canon", "path_to_unique", "unique_paths", "multiplicity", "slot_out"):
        assert np.array_equal(got[key], want[key]), key


# =========================================================================================================
# ss_gather_unique_paths
# =========================================================================================================
@pytest.mark.parametrize("n,frac", [(0, 0.0), (1, 1.0), (5, 0.0), (777, 0.5), (4096, 1.0), (4097, 0.9), (50000, 0.7)])
def test_gather_unique_paths_bit_exact(n, frac):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(n + 3)
    U = int(round(n * frac))
    uniq = np.sort(rng.choice(n, size=U, replace=False)).astype(np.int32) if n else np.zeros(0, np.int32)
    up = np.concatenate([uniq, rng.integers(0, max(n, 1), size=n - U).astype(np.int32)])
    q_len = rng.integers(0, 130, size=n).astype(np.int32)
    q_off = (np.concatenate([[0], np.cumsum(q_len.astype(np.int64))]) + 7).astype(np.int64)
    leaf = rng.integers(0, 1 << 20, size=n).astype(np.int32)
    want = oracle.gather_unique(up, U, n, leaf, q_len, q_off)

    def t(a):
        return torch.from_numpy(a).to(dev) if a.size else torch.zeros(1, dtype=torch.from_numpy(a).dtype, device=dev)
    u_leaf = torch.full((max(n, 1),), 123, dtype=torch.int32, device=dev)
    u_q_len = torch.full((max(n, 1),), 123, dtype=torch.int32, device=dev)
    u_q_src = torch.full((max(n, 1),), 123, dtype=torch.int64, device=dev)
    u_q_off = torch.full((n + 1,), 123, dtype=torch.int64, device=dev)
    num_unique = torch.tensor([U], dtype=torch.int32, device=dev)
    for _ in range(2):                                     # twice: no state between calls
        B.ss_gather_unique_paths(t(up), num_unique, n, t(leaf), t(q_len), t(q_off), u_leaf, u_q_len, u_q_off, u_q_src)
        torch.cuda.synchronize()
        assert np.array_equal(u_leaf[:n].cpu().numpy(), want["u_leaf"])
        assert np.array_equal(u_q_len[:n].cpu().numpy(), want["u_q_len"])
        assert np.array_equal(u_q_src[:n].cpu().numpy(), want["u_q_src"])
        assert np.array_equal(u_q_off.cpu().numpy(), want["u_q_offsets"])


@pytest.mark.parametrize("mode,flags", MODES[:2])
def test_attention_score_jumps_between_tiles(mode, flags):
    """Scores that leap by far more than the lazy-rescale threshold from one key tile to a later one (the K rows of
    some pages are scaled up and the softmax scale is 1): the tensor-core kernels keep a reference maximum that lags
    behind the data and must fall back to their exact path; results still match the fp64 oracle.  With such scores
    the softmax is nearly one-hot, so the output is compared relative to the magnitude of V."""
    w = synth.build_tree_workload("jump", 11, 8, 2, [1024], [4], 1, (300, 700),
                                  lambda i, n, rng: 1 if i % 2 else 40, poison=False)
    pool = w.kv_pool.clone()                                   # [page][2][Hkv][16][128]
    pages = np.unique(w.node_pages)
    rng = np.random.default_rng(3)
    hot = rng.choice(pages, size=max(1, len(pages) // 7), replace=False)
    pool[torch.from_numpy(hot).long(), 0] *= 6.0               # K of some pages: raw scores up to several hundred
    w.kv_pool = pool
    r, ref = attention_only(w, flags, sm_scale=1.0)
    o_ref, l_ref = oracle.tree_attention_workload(w, paths=ref["unique_paths"], sm_scale=1.0)
    assert np.isfinite(r["out"]).all()
    assert np.abs(r["out"] - o_ref).max() <= 4e-2              # |V| up to ~4: bf16 output rounding alone is 1.6e-2
    fin = np.isfinite(l_ref)
    # lse is a raw score here (hundreds): compare relative to its size
    assert np.abs(r["lse"][fin] - l_ref[fin]).max() <= 2e-3 * max(1.0, np.abs(l_ref[fin]).max())


def test_attention_pool_blocks_off_the_8_row_grid():
    """A K / V pool whose (page, head) blocks are 17 rows apart (strides that are multiples of 128 elements, as the
    interface asks, but not of 8 rows): the default tile kernel's one-copy-per-block path cannot address it and the
    call must take the other tensor-core kernel, with the same results."""
    name, Hq, Hkv, levels, fanout, problems, leaf, qfn, dup = SHAPES[1]
    w = synth.build_tree_workload(name, 4321, Hq, Hkv, levels, fanout, problems, leaf, qfn, dup_frac=dup)
    pipe = DevicePipeline(w, DEV, attn_flags=B.SS_FLAG_VALIDATE)
    pool = pipe.kv_pool                                         # [page][2][Hkv][16][128]
    padded = torch.zeros((pool.shape[0], 2, Hkv, 17, 128), dtype=torch.bfloat16, device=pool.device)
    padded[:, :, :, :16] = pool
    padded[:, :, :, 16] = float("nan")                          # the padding row must never be read
    d = pipe.desc
    blk = Hkv * 17 * 128
    d.k_pool = padded.data_ptr()
    d.v_pool = padded.data_ptr() + blk * 2
    d.kv_page_stride, d.kv_head_stride, d.kv_token_stride = 2 * blk, 17 * 128, 128
    pipe.attn_ws = B.alloc_workspace(B.ss_tree_attention_workspace_bytes(d), pool.device)
    pipe.dedup()
    pipe.compact_unique()
    pipe.attention()
    r = pipe.results()
    ref = oracle.dedup(w.tok_ids, w.tok_offsets, w.ctx_key, w.slot_in)
    check_attention(r, w, ref, max_paths=64)
