"""kvcrush_signature_static: the signature stage for hosts that cannot give the library device
memory (an engine that owns the whole pool and bans cudaMalloc on its hot path, a callback that
must not cause the device-wide synchronisation an allocation implies).  Its threshold scratch is
a fixed array inside the library, so the checks are: same bits as kvcrush_signature, twice in a
row with different inputs (the array keeps the previous call's thresholds and must not leak
them), and a clean refusal when the problem needs more thresholds than the array holds.

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test."""
import numpy as np
import pytest

from paper_2503_00022_b200 import inputs

pytestmark = pytest.mark.gpu


def _run_both(B, Hq, seqlens, n_layers, keep, seed):
    import torch
    dev = torch.device("cuda:0")
    T = int(sum(seqlens))
    cu = np.concatenate([[0], np.cumsum(seqlens)])
    scores = np.zeros((n_layers, Hq, T), dtype=np.float32)
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            scores[l, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, seed + 31 * l + s, tie_levels=3 if s % 2 else 0)
    prob = B.Problem(n_layers, Hq, Hq, 16, seqlens, device=dev)
    d_scores = torch.from_numpy(scores).to(dev)
    d_keep = torch.from_numpy(np.asarray(keep, dtype=np.int32).reshape(n_layers, len(seqlens))).to(dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    W = (Hq + 31) // 32
    ref = torch.full((n_layers, T, W), -1, dtype=torch.int32, device=dev)
    got = torch.full((n_layers, T, W), -2, dtype=torch.int32, device=dev)
    ws = torch.empty(max(256, B.kvcrush_workspace_size(prob, B.STAGE_SIGNATURE)), dtype=torch.uint8, device=dev)
    B.kvcrush_signature(prob, d_scores, ref, sig_keep=d_keep, workspace=ws, status=status)
    B.kvcrush_signature_static(prob, d_scores, got, d_keep, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    return ref.cpu().numpy(), got.cpu().numpy()


def test_static_signature_matches_workspace_variant_twice():
    from paper_2503_00022_b200 import binding as B, build
    build.build()
    # first call: 2 layers x 3 sequences x 40 heads (two signature words)
    ref, got = _run_both(B, 40, [300, 77, 1025], 2, [[30, 7, 100], [150, 76, 1]], seed=11)
    np.testing.assert_array_equal(got, ref)
    assert (ref[..., 1] != -1).all()                  # every token was written (word 1 holds only 8 head bits)
    # second call straight after, smaller and with other ranks: stale thresholds of call 1 sit in the array
    ref2, got2 = _run_both(B, 32, [512, 640], 1, [[128, 5]], seed=12)
    np.testing.assert_array_equal(got2, ref2)
    # third: degenerate ranks (all ones / all zeros) go through the same scratch
    ref3, got3 = _run_both(B, 8, [64], 1, [[64]], seed=13)
    np.testing.assert_array_equal(got3, ref3)
    assert (got3.view(np.uint32) == 0xFF).all()


def test_static_signature_refuses_problems_beyond_its_array():
    import torch
    from paper_2503_00022_b200 import binding as B, build
    build.build()
    dev = torch.device("cuda:0")
    n_layers, Hq, seqlens = 9, 128, [1] * 57            # 9 * 57 * 128 = 65664 thresholds > 65536
    assert n_layers * len(seqlens) * Hq > B.STATIC_THETA_MAX
    prob = B.Problem(n_layers, Hq, Hq, 16, seqlens, device=dev)
    T = len(seqlens)
    scores = torch.zeros((n_layers, Hq, T), dtype=torch.float32, device=dev)
    sigs = torch.full((n_layers, T, 4), 5, dtype=torch.int32, device=dev)
    keep = torch.ones((n_layers, T), dtype=torch.int32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(B.KvcrushError) as e:
        B.kvcrush_signature_static(prob, scores, sigs, keep, status=status)
    assert e.value.code == B.ERR_STATIC_LIMIT
    assert "built-in scratch" in str(e.value)
    torch.cuda.synchronize()
    assert (sigs == 5).all()                             # nothing ran
