"""Pins for the signature / selection / compaction part of the oracle
(Algorithm 1 thresholding, Algorithm 2 grouping, Sec. 3.2 kept set)."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    """Fixture format: '#' comments; 'key v1 v2 ...' on one line, or a line holding
    only a key followed by rows of values (rows start with a digit)."""
    out, key = {}, None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            parts = line.split()
            if not parts or parts[0].startswith("#"):
                continue
            if parts[0][0].isdigit():
                out[key].append(parts)
            elif len(parts) == 1:
                key = parts[0]
                out[key] = []
            else:
                out[parts[0]] = parts[1:]
    return out


# --- worked example ---------------------------------------------------------

def test_worked_example():
    g = _read_golden("worked_example.txt")
    s = np.asarray([[float(x) for x in row] for row in g["scores"]], dtype=np.float32)
    theta = O.thresholds(s, 2)
    np.testing.assert_array_equal(theta, np.asarray([float(x) for x in g["theta"][0]], dtype=np.float32))
    sig = O.signatures(s, theta)
    assert [int(x) for x in sig[:, 0]] == [int(x, 16) for x in g["signatures"][0]]
    I = O.importance(s, 4)
    np.testing.assert_allclose(I, [float(x) for x in g["importance"][0]], rtol=1e-6)
    assert abs(I.sum() - 24.0) < 1e-5
    a = O.anchor_bits(O.ANCHOR_ALTERNATE, 4)
    assert int(a[0]) == int(g["anchor"][0][0], 16)
    assert list(O.hamming(sig, a, 4)) == [int(x) for x in g["hamming"][0]]
    for b_imp, b_rep, tag in ((2, 2, "2_2"), (2, 1, "2_1")):
        idx, kind = O.select(s, sig, b_imp, b_rep, 4)
        assert list(idx) == [int(x) for x in g["kept_" + tag][0]]
        assert list(kind) == [int(x) for x in g["kind_" + tag][0]]


def test_hamming_identities():
    H = 40
    g = np.random.Generator(np.random.Philox(2))
    sig = g.integers(0, 1 << 32, size=(50, 2), dtype=np.uint64).astype(np.uint32)
    sig[:, 1] &= np.uint32(0xFF)
    mask = np.asarray([0xFFFFFFFF, 0xFF], dtype=np.uint32)
    for i in range(10):
        assert O.hamming(sig[i:i + 1], sig[i], H)[0] == 0
        assert O.hamming(sig[i:i + 1], (~sig[i]) & mask, H)[0] == H
    assert O.hamming(np.asarray([[0x2]], dtype=np.uint32), np.asarray([0xA], dtype=np.uint32), 4)[0] == 1
    assert O.hamming(np.asarray([[0x9]], dtype=np.uint32), np.asarray([0xA], dtype=np.uint32), 4)[0] == 2
    # agrees with python's bit count and obeys the triangle inequality
    for i, j, l in itertools.islice(itertools.permutations(range(12), 3), 200):
        dij = O.hamming(sig[i:i + 1], sig[j], H)[0]
        assert dij == sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(sig[i], sig[j]))
        assert dij <= O.hamming(sig[i:i + 1], sig[l], H)[0] + O.hamming(sig[l:l + 1], sig[j], H)[0]


def test_alternate_anchor_patterns():
    assert int(O.anchor_bits(O.ANCHOR_ALTERNATE, 32)[0]) == 0xAAAAAAAA
    assert int(O.anchor_bits(O.ANCHOR_ALTERNATE, 8)[0]) == 0xAA
    a = O.anchor_bits(O.ANCHOR_ALTERNATE, 40)
    assert [int(x) for x in a] == [0xAAAAAAAA, 0xAA]


def test_mean_anchor_is_majority_with_ties_to_one():
    sig = np.asarray([[0b0011], [0b0101], [0b0001], [0b1001]], dtype=np.uint32)
    # ones per bit: bit0 4, bit1 1, bit2 1, bit3 1 of N=4 -> only bit0 (2*1 < 4)
    assert int(O.anchor_bits(O.ANCHOR_MEAN, 4, sig)[0]) == 0b0001
    sig2 = np.asarray([[0b10], [0b11]], dtype=np.uint32)   # bit0: 1 of 2 -> tie -> 1
    assert int(O.anchor_bits(O.ANCHOR_MEAN, 2, sig2)[0]) == 0b11


# --- thresholds / signatures --------------------------------------------------

@pytest.mark.parametrize("ties", [0, 6])
def test_threshold_keeps_at_least_k_and_exactly_k_without_ties(ties):
    s = inputs.random_scores(12, 300, 5, tie_levels=ties)
    for k in (1, 17, 150, 299):
        theta = O.thresholds(s, k)
        sig = O.signatures(s, theta)
        ones = O.unpack_bits(sig, 12).sum(axis=0)
        assert np.all(ones >= k)
        for h in range(12):
            n_tied = int((s[h] == theta[h]).sum())
            n_above = int((s[h] > theta[h]).sum())
            assert n_above < k <= n_above + n_tied
            assert ones[h] == n_above + n_tied
            if n_tied == 1:
                assert ones[h] == k
    assert O.unpack_bits(O.signatures(s, O.thresholds(s, 300)), 12).all()
    assert O.unpack_bits(O.signatures(s, O.thresholds(s, 1000)), 12).all()
    assert not O.unpack_bits(O.signatures(s, O.thresholds(s, 0)), 12).any()


def test_signature_is_algorithm1_comparison_with_explicit_theta():
    s = inputs.random_scores(40, 64, 8)
    theta = np.linspace(0.1, 2.0, 40).astype(np.float32)
    sig = O.signatures(s, theta)
    assert sig.shape == (64, 2)
    for t in range(64):
        for h in range(40):
            bit = (int(sig[t, h // 32]) >> (h % 32)) & 1
            assert bit == int(s[h, t] >= theta[h])
    assert np.all(sig[:, 1] < (1 << 8))        # unused high bits are zero


# --- importance -----------------------------------------------------------------

def test_importance_brute_force_and_ties():
    s = inputs.random_scores(8, 200, 3, tie_levels=3)
    for Hkv in (8, 2, 1):
        I = O.importance(s, Hkv)
        np.testing.assert_allclose(I, s.astype(np.float64).sum(axis=0), rtol=1e-14)
    I = O.importance(s, 8)
    assert len(np.unique(I)) < 200                 # ties are present
    for b in (0, 1, 50, 200):
        expect = sorted(sorted(range(200), key=lambda t: (-I[t], t))[:b])
        assert list(O.top_important(I, b)) == expect


def test_importance_gqa_order_is_group_by_group():
    # values chosen so that float64 addition order matters
    s = np.asarray([[1e17], [1.0], [-1e17 + 0.0], [1.0]], dtype=np.float32) * np.float32(1.0)
    flat = O.importance(np.abs(s), 4)
    grouped = O.importance(np.abs(s), 2)
    a, b, c, d = (float(np.abs(s[i, 0])) for i in range(4))
    assert flat[0] == ((a + b) + c) + d
    assert grouped[0] == (a + b) + (c + d)


# --- buckets ---------------------------------------------------------------------

def test_bucket_bounds_exhaustive_small():
    for N in range(1, 65):
        for R in range(1, N + 1):
            b = O.bucket_bounds(N, R)
            sizes = np.diff(b)
            assert b[0] == 0 and b[-1] == N and sizes.sum() == N
            assert set(sizes.tolist()) <= {N // R, -(-N // R)}
            assert sizes.min() >= 1
            # closed form: the bucket of sorted rank r
            for r in range(N):
                i = ((r + 1) * R - 1) // N
                assert b[i] <= r < b[i + 1]


# --- representative ------------------------------------------------------------------

def test_representative_equals_exact_rational_centroid_distance():
    g = np.random.Generator(np.random.Philox(4))
    for trial in range(60):
        H = int(g.integers(1, 41))
        m = int(g.integers(1, 12))
        bits = (g.random((m, H)) < g.random()).astype(np.int64)
        sig = np.stack([O.pack_bits(bits[i]) for i in range(m)])
        toks = np.sort(g.choice(1000, size=m, replace=False))
        cent = [Fraction(int(bits[:, h].sum()), m) for h in range(H)]
        l1 = [sum(abs(Fraction(int(bits[i, h])) - cent[h]) for h in range(H)) for i in range(m)]
        l2 = [sum((Fraction(int(bits[i, h])) - cent[h]) ** 2 for h in range(H)) for i in range(m)]
        best_l1 = min(range(m), key=lambda i: (l1[i], toks[i]))
        best_l2 = min(range(m), key=lambda i: (l2[i], toks[i]))
        assert best_l1 == best_l2
        assert O.representative(toks, sig, H) == int(toks[best_l1])


# --- kept set --------------------------------------------------------------------------

@pytest.mark.parametrize("Hq,Hkv,L,b_imp,b_rep,ties,mode", [
    (8, 8, 96, 12, 12, 0, O.ANCHOR_ALTERNATE),
    (32, 8, 257, 32, 33, 4, O.ANCHOR_ALTERNATE),
    (40, 40, 130, 0, 20, 0, O.ANCHOR_MEAN),
    (12, 4, 64, 10, 1, 2, O.ANCHOR_EXPLICIT),
    (4, 4, 50, 5, 44, 0, O.ANCHOR_ALTERNATE),
])
def test_kept_set_invariants(Hq, Hkv, L, b_imp, b_rep, ties, mode):
    s = inputs.random_scores(Hq, L, 31 + L, tie_levels=ties)
    sig = O.signatures(s, O.thresholds(s, b_imp + b_rep))
    explicit = inputs.random_anchor_bits(Hq, 77)
    idx, kind = O.select(s, sig, b_imp, b_rep, Hkv, mode, explicit)
    assert len(idx) == b_imp + b_rep and np.all(np.diff(idx) > 0)
    imp = set(O.top_important(O.importance(s, Hkv), b_imp).tolist())
    reps = set(idx[kind == 1].tolist())
    assert set(idx[kind == 0].tolist()) == imp and len(reps) == b_rep and not (imp & reps)
    # exactly one representative per bucket, rebuilt here from the definitions
    cand = [t for t in range(L) if t not in imp]
    a = O.anchor_bits(mode, Hq, sig[cand], explicit)
    d = O.hamming(sig, a, Hq)
    srt = sorted(cand, key=lambda t: (d[t], t))
    N = len(cand)
    for i in range(b_rep):
        members = set(srt[(i * N) // b_rep:((i + 1) * N) // b_rep])
        assert len(members & reps) == 1


def test_no_representatives_is_plain_top_b():
    s = inputs.random_scores(16, 120, 9)
    sig = O.signatures(s, O.thresholds(s, 30))
    idx, kind = O.select(s, sig, 30, 0, 16)
    tot = s.astype(np.float64).sum(axis=0)
    assert list(idx) == sorted(np.argsort(-tot, kind="stable")[:30].tolist())
    assert not kind.any()


def test_budget_at_least_length_keeps_everything():
    s = inputs.random_scores(4, 10, 1)
    sig = O.signatures(s, O.thresholds(s, 10))
    for b_imp, b_rep in ((5, 5), (8, 8)):
        idx, kind = O.select(s, sig, b_imp, b_rep, 4)
        assert list(idx) == list(range(10)) and not kind.any()


# --- compaction --------------------------------------------------------------------------

def test_compact_is_index_select():
    g = np.random.Generator(np.random.Philox(6))
    cache = g.standard_normal((50, 4, 8)).astype(np.float16)
    idx = np.sort(g.choice(50, size=13, replace=False))
    out = O.compact(cache, idx)
    ref = torch.index_select(torch.from_numpy(cache), 0, torch.from_numpy(idx)).numpy()
    assert out.tobytes() == ref.tobytes()


# --- Eq. 1 and the signature size ratio -------------------------------------------------

def test_eq1_paper_instance_and_size_ratio():
    g = _read_golden("paper_closed_forms.txt")
    v = {k: int(x[0]) for k, x in g.items()}
    b = O.kv_memory_bytes(v["eq1_batch"], v["eq1_layers"], v["eq1_heads"], v["eq1_seq_len"],
                          v["eq1_head_dim"], v["eq1_precision_bytes"])
    assert b == v["eq1_gib"] * 2 ** 30
    assert v["sig_key_values"] * v["sig_key_value_bits"] // v["sig_bits"] == v["sig_ratio"]
    W = O.signatures(inputs.random_scores(32, 4, 1), np.zeros(32, dtype=np.float32)).shape[1]
    assert W * 32 == v["sig_bits"]


# --- whole pass on a tiny sequence ---------------------------------------------------------

def test_compress_sequence_end_to_end_small():
    w = inputs.Workload("tiny", 1, 4, 2, 16, (48,), inputs.FP32, inputs.FP32, 0.25, budget=12, base_seed=5)
    li = inputs.layer_inputs(w, 0)
    r = O.compress_sequence(inputs.widen(li.q, w.qk_dtype), inputs.widen(li.k, w.qk_dtype), 6, 6)
    assert len(r["idx"]) == 12 and np.all(np.diff(r["idx"]) > 0)
    np.testing.assert_allclose(r["colsum"].sum(axis=1), 48.0, rtol=1e-12)
    # sinks (4x key norm) receive most attention, so they are kept as important
    assert set(range(4)) <= set(r["idx"][r["kind"] == 0].tolist())


# --- SnapKV-style pieces: pooling and the forced recent window ----------------------------------

@pytest.mark.parametrize("kernel", [1, 3, 7, 13])
def test_max_pool_matches_library_pooling(kernel):
    s = inputs.random_scores(6, 97, 21)
    out = O.max_pool(s, kernel)
    ref = torch.nn.functional.max_pool1d(torch.from_numpy(s)[None], kernel, stride=1, padding=(kernel - 1) // 2)[0].numpy()
    np.testing.assert_array_equal(out, ref)
    assert np.all(out >= s)
    if kernel == 1:
        np.testing.assert_array_equal(out, s)


def test_keep_recent_forces_the_window_into_the_important_set():
    s = inputs.random_scores(8, 120, 23)
    s[:, -10:] *= 1e-3                               # the recent tokens would otherwise lose
    sig = O.signatures(s, O.thresholds(s, 30))
    idx0, _ = O.select(s, sig, 20, 10, 8)
    assert not set(range(110, 120)) <= set(idx0.tolist())
    idx, kind = O.select(s, sig, 20, 10, 8, keep_recent=10)
    assert len(idx) == 30 and set(range(110, 120)) <= set(idx[kind == 0].tolist())
    # the other 10 important tokens are the best of the rest
    I = O.importance(s, 8)
    rest = sorted(sorted(range(110), key=lambda t: (-I[t], t))[:10])
    assert sorted(set(idx[kind == 0].tolist()) - set(range(110, 120))) == rest
    # more recent tokens than the important budget: the lowest indices of the window win the ties
    idx2, kind2 = O.select(s, sig, 4, 3, 8, keep_recent=10)
    assert sorted(idx2[kind2 == 0].tolist()) == [110, 111, 112, 113]


def test_keep_initial_and_recent_equal_selection_on_raised_scores():
    """Tokens kept by decree behave like tokens whose scores beat everything: the pinned routine run on
    scores with those columns raised (signatures unchanged) gives the same kept set."""
    s = inputs.random_scores(8, 150, 29, tie_levels=2)
    s[:, :6] *= 1e-3                                  # the initial tokens would otherwise lose
    sig = O.signatures(s, O.thresholds(s, 40))
    raised = s.copy()
    raised[:, :6] = 1e6
    raised[:, -9:] = 1e6
    for b_imp, b_rep in ((25, 15), (15, 25), (40, 0)):
        want = O.select(raised, sig, b_imp, b_rep, 4)
        got = O.select(s, sig, b_imp, b_rep, 4, keep_recent=9, keep_initial=6)
        np.testing.assert_array_equal(got[0], want[0])
        np.testing.assert_array_equal(got[1], want[1])
        assert set(range(6)) | set(range(141, 150)) <= set(got[0][got[1] == 0].tolist())
    # more forced tokens than places: the lowest indices win (initial tokens first)
    idx, kind = O.select(s, sig, 8, 4, 4, keep_recent=9, keep_initial=6)
    assert sorted(idx[kind == 0].tolist()) == [0, 1, 2, 3, 4, 5, 141, 142]
