"""GPU parity of the decode step of the cumulative attention (Sec. 2.3 / 4.1.1: H2O keeps summing attention weights
while tokens are generated): running scores plus one new query's softmax row, within 1e-5 + 2e-3*|oracle|."""
import numpy as np
import pytest

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs
import kvc_testlib as TL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2503_00022_b200 import binding, build
    build.build()
    binding.lib()
    return binding


@pytest.mark.parametrize("dtype,D,Hq,Hkv,seqlens", [
    (inputs.BF16, 128, 8, 2, (700, 1, 129, 2100)),
    (inputs.FP16, 96, 4, 4, (333, 64)),
    (inputs.FP32, 64, 6, 3, (257, 31, 1000)),
    (inputs.BF16, 256, 2, 1, (40,)),
])
def test_decode_update_matches_oracle(B, dtype, D, Hq, Hkv, seqlens):
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload("dec", 2, Hq, Hkv, D, seqlens, dtype, dtype, 0.25, base_seed=140 + D)
    lis, q, k, _, _ = TL.stack_layers(w, range(2), with_cache=False)
    cu = w.cu_seqlens
    last = np.asarray([int(cu[s + 1]) - 1 for s in range(len(seqlens))])
    q_new = np.ascontiguousarray(q[:, last])                                   # [layers, n_seqs, Hq, D]: the new queries
    g = np.random.Generator(np.random.Philox(5))
    base = g.random((2, Hq, w.total_tokens)).astype(np.float32) * 3.0
    prob = B.Problem(2, Hq, Hkv, D, seqlens, device=dev)
    scores = torch.from_numpy(base.copy()).to(dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_score_decode(prob, TL.torch_storage(q_new, dtype, dev), TL.torch_storage(k, dtype, dev), scores, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    got = scores.cpu().numpy()
    for l in range(2):
        for s, L in enumerate(seqlens):
            a, b = int(cu[s]), int(cu[s + 1])
            want = O.decode_update(base[l][:, a:b].astype(np.float64), inputs.widen(q_new[l, s], dtype),
                                   inputs.widen(k[l, a:b], dtype))
            inc_g, inc_o = got[l][:, a:b].astype(np.float64) - base[l][:, a:b], want - base[l][:, a:b]
            # the running value was rounded to float32 after the add: allow its half ulp on top of the tolerance
            assert (np.abs(inc_g - inc_o) <= 1e-5 + 2e-3 * np.abs(inc_o) + 2.5e-7 * np.abs(want)).all(), (l, s)
            np.testing.assert_allclose(inc_g.sum(axis=1), 1.0, rtol=1e-3)


def test_prefill_then_decode_rebuilds_the_column_sums(B):
    """Scores of a 600-token prompt from the tensor-core sweeps, then 8 decode steps: the running scores equal the
    column sums of the 608-token causal attention."""
    import torch
    dev = torch.device("cuda:0")
    L0, n_dec, Hq, Hkv, D = 600, 8, 4, 2, 128
    w = inputs.Workload("predec", 1, Hq, Hkv, D, (L0 + n_dec,), inputs.BF16, inputs.BF16, 0.25, base_seed=150)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    running = torch.zeros((1, Hq, L0 + n_dec), dtype=torch.float32, device=dev)
    prob0 = B.Problem(1, Hq, Hkv, D, (L0,), device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob0, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    pre = torch.empty((1, Hq, L0), dtype=torch.float32, device=dev)
    B.kvcrush_score(prob0, dq[:, :L0], dk[:, :L0], pre, workspace=ws, status=status)
    running[:, :, :L0] = pre
    for j in range(L0, L0 + n_dec):
        prob = B.Problem(1, Hq, Hkv, D, (j + 1,), device=dev)
        view = running[:, :, : j + 1].contiguous()
        B.kvcrush_score_decode(prob, dq[:, j:j + 1], dk[:, : j + 1], view, status=status)
        running[:, :, : j + 1] = view
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    c, _ = O.scores(inputs.widen(lis[0].q, w.qk_dtype), inputs.widen(lis[0].k, w.qk_dtype), True)
    assert TL.within_score_tolerance(running.cpu().numpy()[0], c).all()
