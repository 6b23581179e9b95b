"""Pins of the oracle's clustering baseline (k-means in the place of Algorithm 2's grouping; ablation
"KMeans vs KVCrush", Fig. 3).  CPU only."""
import os
from fractions import Fraction

import numpy as np

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _fixture(name):
    out, key = {}, None
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line[0].isalpha() or line[0] == "_":
            key = line
            out[key] = []
        else:
            out[key].append(line.split())
    return out


def _worked_inputs():
    fx = _fixture("worked_example.txt")
    scores = np.asarray(fx["scores"], dtype=np.float32)
    sig = np.asarray([[int(x, 16)] for x in fx["signatures"][0]], dtype=np.uint32)
    return scores, sig


def test_hand_worked_kmeans_example():
    fx = _fixture("worked_example_kmeans.txt")
    scores, sig = _worked_inputs()
    kept, kind = O.kmeans_select(scores, sig, 2, 2, 4, iterations=int(fx["iterations"][0][0]))
    assert kept.tolist() == [int(x) for x in fx["kept"][0]]
    assert kind.tolist() == [int(x) for x in fx["kind"][0]]
    kept0, _ = O.kmeans_select(scores, sig, 2, 2, 4, iterations=0)
    assert kept0.tolist() == [int(x) for x in fx["kept_0_iterations"][0]]
    # more iterations change nothing once the assignment is stable
    kept9, _ = O.kmeans_select(scores, sig, 2, 2, 4, iterations=9)
    assert kept9.tolist() == kept.tolist()


def test_assignment_is_the_nearest_centroid_in_exact_rationals():
    rng = np.random.default_rng(5)
    for H, N, k in ((8, 40, 5), (33, 60, 7)):
        bits = (rng.random((N, H)) < 0.3).astype(np.int64)
        m = rng.integers(1, 9, size=k)
        cnt = np.stack([rng.integers(0, m[c] + 1, size=H) for c in range(k)])
        got = O.kmeans_assign(bits, cnt, m)
        for t in range(N):
            d = [sum((Fraction(int(bits[t, h])) - Fraction(int(cnt[c, h]), int(m[c]))) ** 2 for h in range(H)) for c in range(k)]
            assert got[t] == min(range(k), key=lambda c: (d[c], c))


def _inertia(bits, cnt, m, assign):
    return sum(sum((Fraction(int(bits[t, h])) - Fraction(int(cnt[assign[t], h]), int(m[assign[t]]))) ** 2
                   for h in range(bits.shape[1])) for t in range(bits.shape[0]))


def test_lloyd_iterations_never_increase_the_within_cluster_sum_of_squares():
    # the classical invariant of Lloyd's algorithm, checked on the oracle's own assign / update steps
    rng = np.random.default_rng(9)
    H, N, k = 6, 50, 6
    bits = (rng.random((N, H)) < 0.4).astype(np.int64)
    cnt = bits[[(i * N) // k for i in range(k)]].copy()
    m = np.ones(k, dtype=np.int64)
    last = None
    for _ in range(6):
        assign = O.kmeans_assign(bits, cnt, m)
        cur = _inertia(bits, cnt, m, assign)
        assert last is None or cur <= last
        for c in range(k):
            mem = assign == c
            if mem.any():
                cnt[c], m[c] = bits[mem].sum(axis=0), int(mem.sum())
        after = _inertia(bits, cnt, m, assign)
        assert after <= cur
        last = after


def test_one_cluster_reduces_to_the_pinned_centroid_representative():
    # k = 1: after one iteration the centroid is the mean of all grouped tokens and the representative is
    # Algorithm 2's "closest to the centroid" over one bucket holding them all
    for seed in (1, 2, 3):
        Hq, L = 8, 40
        s32 = inputs.random_scores(Hq, L, seed)
        sig = O.signatures(s32, O.thresholds(s32, 10))
        kept, kind = O.kmeans_select(s32, sig, 5, 1, Hq, iterations=3)
        imp = O.top_important(O.importance(s32, Hq), 5)
        cand = np.setdiff1d(np.arange(L), imp)
        rep = O.representative(cand, sig[cand], Hq)
        assert kept.tolist() == sorted(imp.tolist() + [rep])
        assert kind[kept.tolist().index(rep)] == 1 and kind.sum() == 1


def test_kept_set_invariants_and_empty_clusters():
    for seed, Hq, L, b_imp, b_rep, it in ((4, 8, 64, 8, 8, 4), (5, 4, 90, 10, 30, 3), (6, 40, 70, 0, 12, 2)):
        s32 = inputs.random_scores(Hq, L, seed, tie_levels=3)
        sig = O.signatures(s32, O.thresholds(s32, b_imp + b_rep))
        kept, kind = O.kmeans_select(s32, sig, b_imp, b_rep, Hq, iterations=it)
        assert kept.shape[0] == b_imp + b_rep and np.all(np.diff(kept) > 0)
        imp = O.top_important(O.importance(s32, Hq), b_imp)
        assert set(imp.tolist()) <= set(kept.tolist())
        assert not (set(kept[kind == 1].tolist()) & set(imp.tolist()))
    # identical vectors: every token falls into cluster 0, the other clusters stay empty, and their budget goes
    # to the most important of the remaining tokens
    Hq, L = 4, 12
    s32 = np.tile(np.linspace(1.0, 2.0, L, dtype=np.float32), (Hq, 1))
    sig = np.zeros((L, 1), dtype=np.uint32)
    kept, kind = O.kmeans_select(s32, sig, 2, 3, Hq, iterations=2)
    # important: 11, 10; grouped 0..9 all identical -> one representative (token 0, lowest index) + fill 9, 8
    assert kept.tolist() == [0, 8, 9, 10, 11] and kind.tolist() == [1, 0, 0, 0, 0]
    # a budget that covers the sequence keeps everything
    kept, kind = O.kmeans_select(s32, sig, 6, 6, Hq)
    assert kept.tolist() == list(range(L)) and not kind.any()
