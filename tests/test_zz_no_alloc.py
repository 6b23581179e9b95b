"""kvcrush_signature_static: the signature stage for hosts that cannot give the library device
memory (an engine that owns the whole pool and bans cudaMalloc on its hot path, a callback that
must not cause the device-wide synchronisation an allocation implies).  Its threshold scratch is
a fixed array inside the library, so the checks are: same bits as kvcrush_signature and as the
CPU oracle, several times in a row with different inputs (the array keeps the previous call's
thresholds and must not leak them), no change of the device's free memory across a call once the
array's address is known, and a clean refusal when the problem needs more thresholds than the
array holds.

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test."""
import numpy as np
import pytest

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs

pytestmark = pytest.mark.gpu


def _run_both(B, Hq, seqlens, n_layers, keep, seed, static_first=False, expect_no_allocation=False):
    """Signatures of the same scores from kvcrush_signature (caller's workspace) and kvcrush_signature_static
    (the library's own array), plus the CPU oracle's for the same float32 scores."""
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
    keep = np.asarray(keep, dtype=np.int32).reshape(n_layers, len(seqlens))
    d_keep = torch.from_numpy(keep).to(dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    W = (Hq + 31) // 32
    ref = torch.full((n_layers, T, W), -1, dtype=torch.int32, device=dev)
    got = torch.full((n_layers, T, W), -2, dtype=torch.int32, device=dev)
    ws = torch.empty(max(256, B.kvcrush_workspace_size(prob, B.STAGE_SIGNATURE)), dtype=torch.uint8, device=dev)

    def with_workspace():
        B.kvcrush_signature(prob, d_scores, ref, sig_keep=d_keep, workspace=ws, status=status)

    def without():
        # every buffer exists already and the binding only forwards pointers, so whatever the device's free
        # memory does between the two readings is the entry point's doing
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dev)[0]
        B.kvcrush_signature_static(prob, d_scores, got, d_keep, status=status)
        torch.cuda.synchronize()
        if expect_no_allocation:
            assert torch.cuda.mem_get_info(dev)[0] == free_before

    for fn in ((without, with_workspace) if static_first else (with_workspace, without)):
        fn()
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    want = np.zeros((n_layers, T, W), dtype=np.uint32)
    for l in range(n_layers):
        for s in range(len(seqlens)):
            s32 = np.ascontiguousarray(scores[l][:, cu[s]:cu[s + 1]])
            want[l, cu[s]:cu[s + 1]] = O.signatures(s32, O.thresholds(s32, int(keep[l, s])))
    return ref.cpu().numpy(), got.cpu().numpy(), want.view(np.int32)


def test_static_signature_matches_workspace_variant_and_the_oracle_twice():
    from paper_2503_00022_b200 import binding as B, build
    build.build()
    # first call: 2 layers x 3 sequences x 40 heads (two signature words); it also looks the array's address up
    ref, got, want = _run_both(B, 40, [300, 77, 1025], 2, [[30, 7, 100], [150, 76, 1]], seed=11)
    np.testing.assert_array_equal(got, ref)
    np.testing.assert_array_equal(got, want)
    assert (ref[..., 1] != -1).all()                  # every token was written (word 1 holds only 8 head bits)
    # second call straight after, smaller, with other ranks and BEFORE the workspace variant: stale thresholds of
    # call 1 sit in the array, the address comes from the cache, and the device's free memory must not move
    ref2, got2, want2 = _run_both(B, 32, [512, 640], 1, [[128, 5]], seed=12, static_first=True, expect_no_allocation=True)
    np.testing.assert_array_equal(got2, ref2)
    np.testing.assert_array_equal(got2, want2)
    # third: degenerate ranks (all ones / all zeros) go through the same scratch
    ref3, got3, want3 = _run_both(B, 8, [64], 1, [[64]], seed=13, expect_no_allocation=True)
    np.testing.assert_array_equal(got3, ref3)
    np.testing.assert_array_equal(got3, want3)
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
