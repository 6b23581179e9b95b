"""GPU parity of the SnapKV-style importance pieces (Sec. 2.3 / 4.1.1 of the paper name them: an observation
window of the final prompt tokens, max pooling over neighbouring scores, the window itself kept):
windowed scores within 1e-5 + 2e-3*|oracle|, pooling and selection bit-exact."""
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


def _dev():
    import torch
    return torch.device("cuda:0")


CASES = [
    # (workload, window)
    (inputs.Workload("win_tc_1k", 1, 4, 2, 128, (1000,), inputs.BF16, inputs.BF16, 0.25, base_seed=61), 64),
    (inputs.Workload("win_tc_ragged", 2, 4, 4, 128, (700, 31, 257, 1300), inputs.BF16, inputs.BF16, 0.25, base_seed=62), 200),
    (inputs.Workload("win_tc_d64", 1, 2, 1, 64, (513, 900), inputs.BF16, inputs.BF16, 0.25, base_seed=63), 1),
    (inputs.Workload("win_tc_wide", 1, 2, 2, 128, (300, 640), inputs.BF16, inputs.BF16, 0.25, base_seed=64), 5000),
    (inputs.Workload("win_tc_noncausal", 1, 2, 2, 128, (333, 520), inputs.BF16, inputs.BF16, 0.25, base_seed=65, causal=False), 130),
    (inputs.Workload("win_simt_fp32", 1, 4, 4, 64, (400, 90), inputs.FP32, inputs.FP32, 0.25, base_seed=66), 48),
]


@pytest.mark.parametrize("w,window", CASES, ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_windowed_scores_match_oracle(B, w, window):
    import torch
    dev = _dev()
    lis, q, k, _, _ = TL.stack_layers(w, range(w.n_layers), with_cache=False)
    prob = B.Problem(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, causal=w.causal, device=dev,
                     query_window=window)
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    T = w.total_tokens
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    impls = [B.SCORE_SIMT] if w.qk_dtype == inputs.FP32 else [B.SCORE_TENSOR, B.SCORE_SIMT]
    cu = w.cu_seqlens
    for impl in impls:
        scores = torch.full((w.n_layers, w.n_q_heads, T), -1.0, dtype=torch.float32, device=dev)
        lse = torch.full_like(scores, 7.0)
        B.kvcrush_score(prob, dq, dk, scores, lse_out=lse, impl=impl, workspace=ws, status=status)
        norm = torch.empty_like(scores)
        B.kvcrush_score(prob, dq, dk, norm, normalize=True, impl=impl, workspace=ws, status=status)
        torch.cuda.synchronize()
        assert status.cpu().tolist()[0] == 0
        g, gl, gn = scores.cpu().numpy(), lse.cpu().numpy(), norm.cpu().numpy()
        for l, li in enumerate(lis):
            for s, L in enumerate(w.seqlens):
                a, b = int(cu[s]), int(cu[s + 1])
                j0 = max(0, L - window)
                c, ol = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), w.causal,
                                 rows=(j0, L))
                ok = TL.within_score_tolerance(g[l][:, a:b], c)
                assert ok.all(), (w.name, impl, l, s, np.argwhere(~ok)[:4])
                np.testing.assert_allclose(gl[l][:, a + j0:b], ol[:, j0:], rtol=0, atol=3e-4)
                np.testing.assert_allclose(gn[l][:, a:b] * (L - j0), g[l][:, a:b], rtol=1e-5, atol=1e-7)
                np.testing.assert_allclose(g[l][:, a:b].astype(np.float64).sum(axis=1), float(L - j0), rtol=2e-4)


@pytest.mark.parametrize("kernel", [1, 3, 7, 33])
def test_pooling_is_bit_exact(B, kernel):
    import torch
    dev = _dev()
    seqlens, Hq, n_layers = [300, 1, 17, 1025], 12, 2
    T = sum(seqlens)
    cu = np.concatenate([[0], np.cumsum(seqlens)])
    scores = np.zeros((n_layers, Hq, T), dtype=np.float32)
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            scores[l, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, 70 + 5 * l + s)
    prob = B.Problem(n_layers, Hq, Hq, 16, seqlens, device=dev)
    out = torch.full((n_layers, Hq, T), -3.0, dtype=torch.float32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_pool_scores(prob, torch.from_numpy(scores).to(dev), kernel, out, status=status)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for l in range(n_layers):
        for s in range(len(seqlens)):
            np.testing.assert_array_equal(got[l][:, cu[s]:cu[s + 1]], O.max_pool(scores[l][:, cu[s]:cu[s + 1]], kernel))


@pytest.mark.parametrize("keep_recent,budgets", [(16, [(40, 30), (20, 10)]), (64, [(10, 5), (64, 64)]), (1, [(1, 1), (0, 9)])])
def test_keep_recent_selection_is_bit_exact(B, keep_recent, budgets):
    import torch
    dev = _dev()
    seqlens, Hq, Hkv = [500, 333], 32, 8
    T = sum(seqlens)
    cu = np.concatenate([[0], np.cumsum(seqlens)])
    scores = np.zeros((1, Hq, T), dtype=np.float32)
    for s, L in enumerate(seqlens):
        scores[0, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, 90 + s, tie_levels=3 * s)
    b_imp = np.asarray([b[0] for b in budgets], dtype=np.int32)
    b_rep = np.asarray([b[1] for b in budgets], dtype=np.int32)
    prob = B.Problem(1, Hq, Hkv, 16, seqlens, device=dev)
    cp = B.CompressionPass(prob, b_imp[None], b_rep[None], keep_recent=keep_recent)
    ds = torch.from_numpy(scores).to(dev)
    cp.signature(ds)
    cp.select(ds)
    torch.cuda.synchronize()
    cp.check_status()
    for s, L in enumerate(seqlens):
        s32 = np.ascontiguousarray(scores[0][:, cu[s]:cu[s + 1]])
        sig = O.signatures(s32, O.thresholds(s32, int(b_imp[s] + b_rep[s])))
        idx, kind = O.select(s32, sig, int(b_imp[s]), int(b_rep[s]), Hkv, keep_recent=keep_recent)
        np.testing.assert_array_equal(cp.kept(0, s), idx.astype(np.int32))
        lo, hi = int(cp.cu_kept_host[s]), int(cp.cu_kept_host[s + 1])
        np.testing.assert_array_equal(cp.kind[lo:hi].cpu().numpy(), kind)


def test_snapkv_style_pass_end_to_end(B):
    """Window scores -> pooling -> signature -> selection with the window kept -> compaction."""
    import torch
    dev = _dev()
    w = inputs.Workload("snap", 2, 8, 2, 128, (900, 400), inputs.BF16, inputs.FP16, 0.25, base_seed=67)
    window, kernel = 32, 7
    lis, q, k, kc, vc = TL.stack_layers(w, range(2))
    prob = B.Problem(2, 8, 2, 128, w.seqlens, device=dev, query_window=window)
    b_imp, b_rep = w.budgets()
    cp = B.CompressionPass(prob, b_imp[None], b_rep[None], cache_dtype=torch.float16, pool_kernel=kernel, keep_recent=window)
    cp.run(TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev),
           TL.torch_storage(kc, w.cache_dtype, dev), TL.torch_storage(vc, w.cache_dtype, dev))
    torch.cuda.synchronize()
    cp.check_status()
    g = cp.scores.cpu().numpy()
    gp = cp.pooled.cpu().numpy()
    cu = w.cu_seqlens
    for l, li in enumerate(lis):
        for s, L in enumerate(w.seqlens):
            a, b = int(cu[s]), int(cu[s + 1])
            c, _ = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), True,
                            rows=(L - window, L))
            assert TL.within_score_tolerance(g[l][:, a:b], c).all()
            pooled = O.max_pool(np.ascontiguousarray(g[l][:, a:b]), kernel)
            np.testing.assert_array_equal(gp[l][:, a:b], pooled)
            sig = O.signatures(pooled, O.thresholds(pooled, int(b_imp[s] + b_rep[s])))
            idx, kind = O.select(pooled, sig, int(b_imp[s]), int(b_rep[s]), 2, keep_recent=window)
            np.testing.assert_array_equal(cp.kept(l, s), idx.astype(np.int32))
            assert set(range(L - window, L)) <= set(idx[kind == 0].tolist())
            seg = l * w.n_seqs + s
            lo = int(cp.cu_kept_host[seg]) - int(cp.cu_kept_host[l * w.n_seqs])
            got = cp.k_out[l, lo:lo + len(idx)].cpu().numpy()
            assert got.tobytes() == O.compact(li.k_cache[a:b], idx).tobytes()
