"""Pins for the score part of the oracle (Algorithm 1: softmax attention and its
per-token sums).  None of these re-types the oracle's own loop: they compare it
with explicit matrices, closed forms, invariants and a library routine."""
import numpy as np
import pytest
import torch

from oracle import kvcrush_oracle as O


def _rand_qk(L, Hq, Hkv, D, seed):
    g = np.random.Generator(np.random.Philox(seed))
    q = g.standard_normal((L, Hq, D))
    k = g.standard_normal((L, Hkv, D))
    k[: min(4, L)] *= 4.0
    return q, k


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("L,Hq,Hkv,D", [(1, 2, 2, 8), (7, 4, 4, 16), (33, 4, 2, 8), (64, 8, 2, 32)])
def test_c_routine_matches_explicit_matrix(L, Hq, Hkv, D, causal):
    q, k = _rand_qk(L, Hq, Hkv, D, 7 + L)
    c, lse = O.scores(q, k, causal)
    np.testing.assert_allclose(c, O.scores_bruteforce(q, k, causal), rtol=1e-12, atol=1e-14)
    # lse against a direct log-sum-exp of the logits
    G = Hq // Hkv
    for h in range(Hq):
        S = (q[:, h] @ k[:, h // G].T) / np.sqrt(D)
        for j in range(L):
            row = S[j, : j + 1] if causal else S[j]
            assert abs(lse[h, j] - np.log(np.exp(row).sum())) < 1e-10


@pytest.mark.parametrize("causal", [True, False])
def test_rows_sum_to_one_and_columns_total_number_of_queries(causal):
    q, k = _rand_qk(48, 4, 2, 16, 11)
    A = O.attention_matrix(q, k, causal)
    # the printed index order of Algorithm 1 (sum over the second index) is a softmax
    # row sum: identically 1, which is why the column sum is the reading used
    np.testing.assert_allclose(A.sum(axis=2), 1.0, rtol=0, atol=1e-12)
    c, _ = O.scores(q, k, causal)
    np.testing.assert_allclose(c.sum(axis=1), 48.0, rtol=1e-12)
    if causal:
        assert np.all(A[:, np.triu_indices(48, 1)[0], np.triu_indices(48, 1)[1]] == 0.0)
        assert np.all(c[:, 0] >= 1.0 - 1e-12)                      # token 0 gets all of query 0
        np.testing.assert_allclose(c[:, -1], A[:, -1, -1], rtol=1e-12)   # last key: one query only


def test_zero_queries_give_harmonic_numbers():
    # Q = 0: every causal row is uniform over its j+1 keys, so c(t) = sum_{j>=t} 1/(j+1) = H_L - H_t
    L, H, D = 40, 3, 8
    q = np.zeros((L, H, D))
    _, k = _rand_qk(L, H, H, D, 3)
    c, lse = O.scores(q, k, True)
    harm = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, L + 1))])
    expect = harm[L] - harm[:L]
    np.testing.assert_allclose(c, np.broadcast_to(expect, (H, L)), rtol=1e-13)
    np.testing.assert_allclose(lse, np.broadcast_to(np.log(np.arange(1, L + 1)), (H, L)), rtol=1e-13, atol=1e-15)
    c_full, _ = O.scores(q, k, False)
    np.testing.assert_allclose(c_full, 1.0, rtol=1e-13)


def test_identical_keys_equal_zero_queries():
    L, H, D = 24, 2, 8
    q, _ = _rand_qk(L, H, H, D, 5)
    k = np.broadcast_to(np.linspace(-1, 1, D), (L, H, D)).copy()
    c, _ = O.scores(q, k, True)
    harm = np.concatenate([[0.0], np.cumsum(1.0 / np.arange(1, L + 1))])
    np.testing.assert_allclose(c, np.broadcast_to(harm[L] - harm[:L], (H, L)), rtol=1e-12)


@pytest.mark.parametrize("causal", [True, False])
def test_matches_library_softmax(causal):
    L, Hq, Hkv, D = 257, 4, 2, 32
    q, k = _rand_qk(L, Hq, Hkv, D, 21)
    c, _ = O.scores(q, k, causal)
    tq = torch.from_numpy(q).permute(1, 0, 2)                              # [Hq, L, D]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    logits = tq @ tk.transpose(1, 2) / np.sqrt(D)
    if causal:
        logits = logits.masked_fill(~torch.tril(torch.ones(L, L, dtype=torch.bool)), float("-inf"))
    ref = torch.softmax(logits, dim=-1).sum(dim=-2).numpy()
    np.testing.assert_allclose(c, ref, rtol=1e-11, atol=1e-13)


def test_gqa_equals_mha_with_repeated_key_heads():
    L, Hq, Hkv, D = 50, 8, 2, 16
    q, k = _rand_qk(L, Hq, Hkv, D, 9)
    c_gqa, _ = O.scores(q, k, True)
    c_mha, _ = O.scores(q, np.repeat(k, Hq // Hkv, axis=1), True)
    np.testing.assert_array_equal(c_gqa, c_mha)


def test_row_range_gives_complete_tail_columns():
    L, Hq, Hkv, D = 90, 4, 2, 16
    q, k = _rand_qk(L, Hq, Hkv, D, 19)
    c, lse = O.scores(q, k, True)
    for j0, j1 in ((60, 90), (0, 90), (33, 34)):
        cp, lp = O.scores(q, k, True, rows=(j0, j1))
        A = O.attention_matrix(q, k, True)
        np.testing.assert_allclose(cp, A[:, j0:j1, :].sum(axis=1), rtol=1e-12, atol=1e-15)
        np.testing.assert_array_equal(lp[:, j0:j1], lse[:, j0:j1])
        if j1 == L:
            np.testing.assert_array_equal(cp[:, j0:], c[:, j0:])       # keys >= j0 are only seen by rows >= j0


def test_scale_and_normalize():
    L, H, D = 20, 2, 8
    q, k = _rand_qk(L, H, H, D, 13)
    c1, _ = O.scores(q, k, True, scale=0.5)
    c2, _ = O.scores(q * 0.5 * np.sqrt(D), k, True)          # default scale 1/sqrt(D)
    np.testing.assert_allclose(c1, c2, rtol=1e-12)
    w, _ = O.scores(q, k, True, normalize=True)
    c, _ = O.scores(q, k, True)
    np.testing.assert_allclose(w * L, c, rtol=1e-15)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, rtol=1e-12)   # Algorithm 1's 1/S makes a distribution


def test_thread_count_does_not_change_result():
    import os
    import subprocess
    import sys
    code = ("import numpy as np, sys; sys.path.insert(0, %r); from oracle import kvcrush_oracle as O;"
            "g=np.random.Generator(np.random.Philox(1)); q=g.standard_normal((64,8,16)); k=g.standard_normal((64,8,16));"
            "c,_=O.scores(q,k,True); sys.stdout.write(c.tobytes().hex())")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for n in ("1", "4"):
        env = dict(os.environ, OMP_NUM_THREADS=n)
        outs.append(subprocess.check_output([sys.executable, "-c", code % root], env=env))
    assert outs[0] == outs[1]


def test_planted_transposition_is_caught():
    # a mistake planted in a copy of the oracle: summing A over keys instead of queries
    q, k = _rand_qk(16, 2, 2, 8, 17)
    A = O.attention_matrix(q, k, True)
    wrong = A.sum(axis=2)
    c, _ = O.scores(q, k, True)
    assert not np.allclose(wrong, c)
    # and a dropped causal mask changes the harmonic closed form
    c_nc, _ = O.scores(np.zeros_like(q), k, False)
    assert not np.allclose(c_nc[0], O.scores(np.zeros_like(q), k, True)[0][0])


def test_decode_update_adds_the_last_row_of_the_attention_matrix():
    L, Hq, Hkv, D = 37, 4, 2, 16
    q, k = _rand_qk(L, Hq, Hkv, D, 31)
    A = O.attention_matrix(q, k, True)                     # [Hq, query, key]
    base = np.arange(Hq * L, dtype=np.float64).reshape(Hq, L) / 7.0
    got = O.decode_update(base, q[L - 1], k)
    np.testing.assert_allclose(got - base, A[:, L - 1, :], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose((got - base).sum(axis=1), 1.0, rtol=1e-12)
    # decoding the whole prompt token by token rebuilds the prefill column sums
    run = np.zeros((Hq, L))
    for j in range(L):
        run[:, : j + 1] = O.decode_update(run[:, : j + 1], q[j], k[: j + 1])
    c, _ = O.scores(q, k, True)
    np.testing.assert_allclose(run, c, rtol=1e-11, atol=1e-13)
    tq = torch.from_numpy(q[L - 1])                        # library softmax
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    ref = torch.softmax((tk @ tq[:, :, None])[:, :, 0] / np.sqrt(D), dim=-1).numpy()
    np.testing.assert_allclose(got - base, ref, rtol=1e-11, atol=1e-14)
