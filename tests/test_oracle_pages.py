"""Pins for the page-granular part of the oracle (Sec. 4.3.4 chunks, Sec. 4.3.5 pages): a hand-worked
example, the reduction to the token-level routine at page size 1, exact rational centroid distances on
page vectors, brute-force page ranking, invariants of the kept set and a library gather."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs
from test_oracle_select import _read_golden


def _sigs_for(scores, keep):
    return O.signatures(scores, O.thresholds(scores, keep))


def test_worked_example_pages():
    g = _read_golden("worked_example_pages.txt")
    s = np.asarray([[float(x) for x in row] for row in g["scores"]], dtype=np.float32)
    theta = O.thresholds(s, 3)
    np.testing.assert_array_equal(theta, np.asarray([float(x) for x in g["theta"][0]], dtype=np.float32))
    sig = O.signatures(s, theta)
    assert [int(x) for x in sig[:, 0]] == [int(x, 16) for x in g["signatures"][0]]
    I = O.importance(s, 2)
    np.testing.assert_allclose(I, [float(x) for x in g["importance"][0]], rtol=1e-6)
    np.testing.assert_allclose(O.page_importance(I, 2), [float(x) for x in g["page_importance"][0]], rtol=1e-6)
    vec = O.page_vectors(sig, 2)
    assert [[int(x) for x in row] for row in vec] == [[int(x, 16) for x in row] for row in g["page_vectors"]]
    a = np.tile(O.anchor_bits(O.ANCHOR_ALTERNATE, 2), 2)
    assert list(O.hamming(vec, a, 64)) == [int(x) for x in g["page_hamming"][0]]
    for b_imp, b_rep, tag in ((1, 1, "1_1"), (1, 2, "1_2")):
        idx, kind = O.select_pages(s, sig, 2, b_imp, b_rep, 2)
        assert list(idx) == [int(x) for x in g["kept_" + tag][0]]
        assert list(kind) == [int(x) for x in g["kind_" + tag][0]]


@pytest.mark.parametrize("Hq,Hkv,L,b_imp,b_rep,ties,mode", [
    (8, 8, 60, 10, 12, 0, 0), (40, 8, 97, 5, 30, 3, 1), (32, 4, 130, 0, 17, 2, 2), (4, 1, 33, 7, 0, 0, 0),
])
def test_page_size_one_is_the_token_level_routine(Hq, Hkv, L, b_imp, b_rep, ties, mode):
    s = inputs.random_scores(Hq, L, 300 + L, tie_levels=ties)
    sig = _sigs_for(s, b_imp + b_rep)
    explicit = inputs.random_anchor_bits(Hq, 9)
    it, kt = O.select(s, sig, b_imp, b_rep, Hkv, mode, explicit)
    ip, kp = O.select_pages(s, sig, 1, b_imp, b_rep, Hkv, mode, explicit)
    np.testing.assert_array_equal(it, ip)
    np.testing.assert_array_equal(kt, kp)


def test_page_importance_is_a_blockwise_sum_and_ranks_like_brute_force():
    g = np.random.Generator(np.random.Philox(5))
    for L, P in ((64, 8), (61, 8), (33, 32), (7, 2), (5, 9)):
        I = g.integers(0, 1 << 20, size=L).astype(np.float64) / 1024.0      # dyadic: every sum is exact
        J = O.page_importance(I, P)
        n_pages = (L + P - 1) // P
        padded = np.zeros(n_pages * P)
        padded[:L] = I
        np.testing.assert_array_equal(J, np.add.reduceat(padded, np.arange(0, n_pages * P, P)))
        assert J.sum() == I.sum()
    # no representatives: the kept pages are the top pages by summed importance, ties to the lower page
    s = inputs.random_scores(8, 100, 77, tie_levels=2)
    sig = _sigs_for(s, 20)
    J = O.page_importance(O.importance(s, 8), 8)
    brute = sorted(sorted(range(len(J)), key=lambda p: (-J[p], p))[:5])
    idx, kind = O.select_pages(s, sig, 8, 5, 0, 8)
    assert list(idx) == brute and not kind.any()


def test_page_vectors_are_the_concatenated_token_vectors():
    g = np.random.Generator(np.random.Philox(6))
    Hq, L, P = 40, 21, 4
    sig = g.integers(0, 1 << 32, size=(L, 2), dtype=np.uint64).astype(np.uint32)
    sig[:, 1] &= np.uint32(0xFF)
    vec = O.page_vectors(sig, P)
    assert vec.shape == (6, 8)
    bits = O.unpack_bits(sig, Hq)                          # [L, Hq]
    for p in range(6):
        for i in range(P):
            t = p * P + i
            for h in range(Hq):
                got = (int(vec[p, i * 2 + h // 32]) >> (h % 32)) & 1
                assert got == (int(bits[t, h]) if t < L else 0)


def test_page_representative_equals_exact_rational_centroid_distance():
    g = np.random.Generator(np.random.Philox(8))
    Hq, P = 5, 3
    for trial in range(40):
        m = int(g.integers(1, 9))
        bits = g.integers(0, 2, size=(m, P, Hq))
        if trial % 4 == 0 and m > 1:
            bits[1] = bits[0]                              # forced tie
        words = np.zeros((m, P), dtype=np.uint32)
        for h in range(Hq):
            words |= (bits[:, :, h].astype(np.uint32) << np.uint32(h))
        pages = np.sort(g.choice(50, size=m, replace=False))
        flat = bits.reshape(m, P * Hq)
        centroid = [Fraction(int(flat[:, j].sum()), m) for j in range(P * Hq)]
        l1 = [sum(abs(Fraction(int(b)) - c) for b, c in zip(row, centroid)) for row in flat]
        l2 = [sum((Fraction(int(b)) - c) ** 2 for b, c in zip(row, centroid)) for row in flat]
        want = min(range(m), key=lambda i: (l1[i], pages[i]))
        assert want == min(range(m), key=lambda i: (l2[i], pages[i]))
        assert O.representative(pages, words, 32 * P) == int(pages[want])


@pytest.mark.parametrize("Hq,Hkv,L,P,b_imp,b_rep,ties,mode", [
    (8, 8, 100, 8, 3, 4, 0, 0), (32, 8, 1000, 32, 4, 9, 2, 0), (40, 40, 517, 8, 10, 20, 3, 1),
    (16, 2, 64, 32, 1, 0, 0, 0), (12, 4, 301, 4, 0, 30, 5, 2), (8, 1, 200, 8, 5, 1, 0, 1),
])
def test_kept_pages_invariants(Hq, Hkv, L, P, b_imp, b_rep, ties, mode):
    s = inputs.random_scores(Hq, L, 40 + L, tie_levels=ties)
    sig = _sigs_for(s, (b_imp + b_rep) * P)
    explicit = inputs.random_anchor_bits(Hq, 4)
    idx, kind = O.select_pages(s, sig, P, b_imp, b_rep, Hkv, mode, explicit)
    n_pages = (L + P - 1) // P
    assert len(idx) == min(n_pages, b_imp + b_rep)
    assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < n_pages
    if b_imp + b_rep < n_pages:
        assert int((kind == 0).sum()) == b_imp and int((kind == 1).sum()) == b_rep
        J = O.page_importance(O.importance(s, Hkv), P)
        assert list(idx[kind == 0]) == sorted(sorted(range(n_pages), key=lambda p: (-J[p], p))[:b_imp])
        # one representative from each bucket of the (d, p) order of the other pages
        vec = O.page_vectors(sig, P)
        cand = np.setdiff1d(np.arange(n_pages), idx[kind == 0])
        if mode == O.ANCHOR_MEAN:
            a = O.anchor_bits(O.ANCHOR_MEAN, 32 * vec.shape[1], vec[cand])
        else:
            a = np.tile(O.anchor_bits(mode, Hq, None, explicit), P)
        d = [sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(vec[p], a)) for p in cand]
        order = [p for _, p in sorted(zip(d, cand.tolist()))]
        bounds = O.bucket_bounds(len(cand), b_rep) if b_rep else []
        reps = set(idx[kind == 1].tolist())
        for i in range(b_rep):
            assert len(reps & set(order[bounds[i]:bounds[i + 1]])) == 1


def test_mean_page_anchor_is_the_per_bit_majority_of_the_grouped_pages():
    s = inputs.random_scores(6, 90, 12)
    sig = _sigs_for(s, 30)
    vec = O.page_vectors(sig, 4)
    cand = np.arange(3, vec.shape[0])
    a = O.anchor_bits(O.ANCHOR_MEAN, 32 * vec.shape[1], vec[cand])
    for w in range(vec.shape[1]):
        for b in range(32):
            ones = sum((int(v[w]) >> b) & 1 for v in vec[cand])
            assert ((int(a[w]) >> b) & 1) == (1 if 2 * ones >= len(cand) else 0)


def test_compact_pages_is_a_padded_library_gather():
    g = np.random.Generator(np.random.Philox(3))
    L, P = 29, 8
    cache = g.standard_normal((L, 2, 4)).astype(np.float16)
    pages = np.asarray([0, 2, 3])
    padded = torch.zeros((32, 2, 4), dtype=torch.float16)
    padded[:L] = torch.from_numpy(cache)
    want = padded.reshape(4, P, 2, 4).index_select(0, torch.from_numpy(pages)).numpy()
    got = O.compact_pages(cache, pages, P)
    assert got.tobytes() == want.tobytes()
    assert not got[2, 5:].any()                            # slots past the end of the sequence


def test_paged_budget_of_table1_keeps_initial_and_recent_pages():
    """Table 1's paged setting: 672 tokens = 32 initial + 512 middle + 128 recent at page size 32, i.e. 1 + 16 + 4
    pages, a quarter of the middle pages chosen as representatives."""
    P, L, Hq = 32, 4000, 8
    s = inputs.random_scores(Hq, L, 51)
    s[:, :P] *= 1e-3
    s[:, -4 * P:] *= 1e-3
    sig = _sigs_for(s, 672)
    idx, kind = O.select_pages(s, sig, P, 17, 4, 8, keep_initial=1, keep_recent=4)
    n_pages = (L + P - 1) // P
    assert len(idx) == 21
    forced = {0} | set(range(n_pages - 4, n_pages))
    assert forced <= set(idx[kind == 0].tolist())
    J = O.page_importance(O.importance(s, 8), P)
    middle = sorted(sorted(set(range(n_pages)) - forced, key=lambda p: (-J[p], p))[:12])
    assert sorted(set(idx[kind == 0].tolist()) - forced) == middle
    # same thing through raised scores and no decree
    raised = s.copy()
    raised[:, :P] = 1e6
    raised[:, (n_pages - 4) * P:] = 1e6
    want = O.select_pages(raised, sig, P, 17, 4, 8)
    np.testing.assert_array_equal(idx, want[0])
    np.testing.assert_array_equal(kind, want[1])
