"""Property tests (hypothesis) of the CPU oracle against brute-force definitions on small random inputs."""
import math

import numpy as np
from hypothesis import given, settings
from hypothesis import strategies as st

import oracle

seqs_st = st.lists(st.tuples(st.integers(0, 2), st.lists(st.integers(0, 2), max_size=4)), min_size=0, max_size=24)


@settings(max_examples=150, deadline=None)
@given(seqs_st)
def test_dedup_equals_pairwise_definition(items):
    ctx = [c for c, _ in items]
    seqs = [s for _, s in items]
    off = np.concatenate([[0], np.cumsum([len(s) for s in seqs])]).astype(np.int64)
    ids = np.asarray([t for s in seqs for t in s], np.int32)
    r = oracle.dedup(ids, off, ctx_key=np.asarray(ctx, np.int64) if items else None)
    canon = []
    for i in range(len(items)):
        canon.append(next(j for j in range(i + 1) if ctx[j] == ctx[i] and seqs[j] == seqs[i]))
    assert list(r["canon"]) == canon
    uniq = [i for i, c in enumerate(canon) if c == i]
    assert list(r["unique_paths"]) == uniq
    assert list(r["multiplicity"]) == [canon.count(u) for u in uniq]


scores_st = st.lists(st.one_of(st.sampled_from([0.0, -0.0, 0.5, 1.0, float("nan"), float("inf"), -1.0]),
                               st.floats(0, 1, width=32)), min_size=0, max_size=20)


def _rank_key(x, i):
    return (1 if math.isnan(x) else 0, 0.0 if math.isnan(x) else -(x + 0.0), i)


@settings(max_examples=150, deadline=None)
@given(scores_st, st.integers(1, 6))
def test_topk_equals_sorted_definition(scores, k):
    sc = np.asarray(scores, np.float32)
    surv, keep = oracle.topk(sc, [0, len(sc)], k)
    order = [i for _, _, i in sorted(_rank_key(float(x), i) for i, x in enumerate(sc))]
    want = order[:k] + [-1] * max(0, k - len(order))
    assert list(surv[0]) == want
    assert list(keep) == [1 if i in order[:k] else 0 for i in range(len(sc))]


@settings(max_examples=150, deadline=None)
@given(scores_st, st.lists(st.booleans(), min_size=20, max_size=20), st.integers(1, 4))
def test_early_prune_rules(scores, ver_bits, k):
    sc = np.asarray(scores, np.float32)
    n = len(sc)
    ver = np.asarray(ver_bits[:n], np.uint8)
    pruned, sel, fin = oracle.early_prune(sc, ver, [0, n], k)
    verified = [i for i in range(n) if ver[i]]
    perfect = [i for i in verified if sc[i] >= 1.0]
    if len(perfect) >= k:                                            # rule 2
        assert fin[0] == 1 and list(sel[0]) == perfect[:k]
        assert [i for i in range(n) if not pruned[i]] == perfect[:k]
    else:
        order = [i for _, _, i in sorted(_rank_key(float(sc[i]), i) for i in verified)]
        assert all(not pruned[i] for i in range(n) if not ver[i])    # rule 1 never touches unverified candidates
        assert [i for i in verified if pruned[i]] == sorted(order[k:]) if len(verified) > k else not pruned.any()
        assert fin[0] == (1 if len(verified) == n else 0)
