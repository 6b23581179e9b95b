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
            # the running value is stored as float32 after the add: one float32 ulp (2^-23) of it on top of the
            # tolerance of the increment
            assert (np.abs(inc_g - inc_o) <= 1e-5 + 2e-3 * np.abs(inc_o) + 2.0 ** -23 * np.abs(want)).all(), (l, s)
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


def test_compact_scores_is_a_gather(B):
    import torch
    dev = torch.device("cuda:0")
    seqlens, Hq, n_layers, P = [100, 37], 6, 2, 8
    T = sum(seqlens)
    g = np.random.Generator(np.random.Philox(8))
    scores = g.random((n_layers, Hq, T)).astype(np.float32)
    prob = B.Problem(n_layers, Hq, 2, 16, seqlens, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    # token level: 3 kept tokens of sequence 0, 2 of sequence 1, per layer
    idx = np.asarray([5, 50, 99, 0, 36, 1, 2, 3, 10, 11], dtype=np.int32)
    cu_kept = np.asarray([0, 3, 5, 8, 10], dtype=np.int32)
    out = torch.full((n_layers, Hq, 7), -1.0, dtype=torch.float32, device=dev)
    B.kvcrush_compact_scores(prob, torch.from_numpy(scores).to(dev), 0, torch.from_numpy(cu_kept).to(dev),
                             torch.from_numpy(idx).to(dev), 10, out, status=status)
    got = out.cpu().numpy()
    np.testing.assert_array_equal(got[0][:, :5], np.concatenate([scores[0][:, [5, 50, 99]], scores[0][:, [100, 136]]], axis=1))
    np.testing.assert_array_equal(got[1][:, :5], np.concatenate([scores[1][:, [1, 2, 3]], scores[1][:, [110, 111]]], axis=1))
    assert (got[:, :, 5:] == -1.0).all()                       # columns past the kept rows are not touched
    # page level: pages {0, 12} of sequence 0 (page 12 holds 4 tokens), page {4} of sequence 1 (5 tokens), layer 0 only
    prob1 = B.Problem(1, Hq, 2, 16, seqlens, device=dev)
    pidx = np.asarray([0, 12, 4], dtype=np.int32)
    pcu = np.asarray([0, 2, 3], dtype=np.int32)
    outp = torch.full((1, Hq, 3 * P), -1.0, dtype=torch.float32, device=dev)
    B.kvcrush_compact_scores(prob1, torch.from_numpy(scores[:1].copy()).to(dev), P, torch.from_numpy(pcu).to(dev),
                             torch.from_numpy(pidx).to(dev), 3, outp, status=status)
    gp = outp.cpu().numpy()[0]
    want = np.zeros((Hq, 3 * P), dtype=np.float32)
    want[:, 0:8] = scores[0][:, 0:8]
    want[:, 8:12] = scores[0][:, 96:100]
    want[:, 16:21] = scores[0][:, 100 + 32:100 + 37]
    np.testing.assert_array_equal(gp, want)


def test_decode_time_paged_eviction_loop(B):
    """Prefill, then decode steps with page-granular eviction whenever the cache outgrows its budget (Table 1's paged
    setting in small: 1 initial page, 4 recent pages, the rest split between important and representative pages).
    Every step is checked against the oracle run on the GPU's own state before the step."""
    import torch
    dev = torch.device("cuda:0")
    n_layers, Hq, Hkv, D, P = 2, 8, 2, 128, 32
    L0, n_dec = 700, 70
    b_imp, b_rep, keep_i, keep_r = 13, 4, 1, 4                   # 17 pages = 544 tokens
    cap = 17 * P + 64
    w = inputs.Workload("loop", n_layers, Hq, Hkv, D, (L0 + n_dec,), inputs.BF16, inputs.BF16, 0.25, base_seed=160)
    lis, q, k, kc, vc = TL.stack_layers(w, range(n_layers))
    dq = TL.torch_storage(q, w.qk_dtype, dev)
    dk_all, dv_all = TL.torch_storage(k, w.qk_dtype, dev), TL.torch_storage(vc, w.cache_dtype, dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)

    # prefill on the whole prompt
    prob = B.Problem(n_layers, Hq, Hkv, D, (L0,), device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    scores = torch.empty((n_layers, Hq, L0), dtype=torch.float32, device=dev)
    B.kvcrush_score(prob, dq[:, :L0], dk_all[:, :L0], scores, workspace=ws, status=status)
    K = dk_all[:, :L0].clone()
    V = dv_all[:, :L0].clone()
    n = L0
    n_evictions = 0
    for step in range(n_dec + 1):
        if n > 17 * P:                                            # over budget: evict down to 17 pages
            prob = B.Problem(n_layers, Hq, Hkv, D, (n,), device=dev)
            cp = B.CompressionPass(prob, np.asarray([[b_imp]]), np.asarray([[b_rep]]), cache_dtype=K.dtype, page_size=P,
                                   keep_initial=keep_i, keep_recent=keep_r)
            host_scores = scores.cpu().numpy()
            cp.signature(scores)
            cp.select(scores)
            cp.compact(K, V)
            new_scores = torch.empty((n_layers, Hq, 17 * P), dtype=torch.float32, device=dev)
            B.kvcrush_compact_scores(prob, scores, P, cp.cu_kept, cp.idx, cp.total_kept, new_scores, status=status)
            torch.cuda.synchronize()
            cp.check_status()
            hK, hV = K.cpu().view(torch.int16).numpy(), V.cpu().view(torch.int16).numpy()
            n_pages = (n + P - 1) // P
            n_new = None
            for l in range(n_layers):
                s32 = np.ascontiguousarray(host_scores[l])
                sig = O.signatures(s32, O.thresholds(s32, (b_imp + b_rep) * P))
                idx, kind = O.select_pages(s32, sig, P, b_imp, b_rep, Hkv, keep_initial=keep_i, keep_recent=keep_r)
                np.testing.assert_array_equal(cp.kept(l, 0), idx.astype(np.int32))
                assert {0} | set(range(n_pages - keep_r, n_pages)) <= set(idx.tolist())
                assert cp.k_out[l].cpu().view(torch.int16).numpy().tobytes() == O.compact_pages(hK[l], idx, P).tobytes()
                assert cp.v_out[l].cpu().view(torch.int16).numpy().tobytes() == O.compact_pages(hV[l], idx, P).tobytes()
                want_sc = np.zeros((Hq, 17 * P), dtype=np.float32)
                for i, p in enumerate(idx):
                    m = min(P, n - int(p) * P)
                    want_sc[:, i * P:i * P + m] = s32[:, int(p) * P:int(p) * P + m]
                np.testing.assert_array_equal(new_scores[l].cpu().numpy(), want_sc)
                n_here = sum(min(P, n - int(p) * P) for p in idx)
                assert n_new in (None, n_here)                    # the last page is kept in every layer
                n_new = n_here
            K, V, scores, n = cp.k_out.clone(), cp.v_out.clone(), new_scores, n_new
            n_evictions += 1
        if step == n_dec:
            break
        # one decode step: the token's key / value join the cache, its query adds an attention row
        j = L0 + step
        if K.shape[1] < n + 1:
            K = torch.cat([K[:, :n], torch.zeros((n_layers, cap, Hkv, D), dtype=K.dtype, device=dev)], dim=1)
            V = torch.cat([V[:, :n], torch.zeros((n_layers, cap, Hkv, D), dtype=V.dtype, device=dev)], dim=1)
        K[:, n] = dk_all[:, j]
        V[:, n] = dv_all[:, j]
        n += 1
        prev = torch.zeros((n_layers, Hq, n), dtype=torch.float32, device=dev)
        prev[:, :, : n - 1] = scores[:, :, : n - 1]
        cur = prev.clone()
        prob = B.Problem(n_layers, Hq, Hkv, D, (n,), device=dev)
        Kn = K[:, :n].contiguous()
        B.kvcrush_score_decode(prob, dq[:, j:j + 1], Kn, cur, status=status)
        torch.cuda.synchronize()
        hp, hc = prev.cpu().numpy().astype(np.float64), cur.cpu().numpy().astype(np.float64)
        hk = Kn.cpu().view(torch.int16).numpy().view(np.uint16)
        for l in range(n_layers):
            want = O.decode_update(hp[l], inputs.widen(q[l, j], w.qk_dtype), inputs.widen(hk[l], w.qk_dtype))
            inc_g, inc_o = hc[l] - hp[l], want - hp[l]
            assert (np.abs(inc_g - inc_o) <= 1e-5 + 2e-3 * np.abs(inc_o) + 2.0 ** -23 * np.abs(want)).all(), (step, l)
        scores = cur
        K, V = K[:, :n], V[:, :n]
    assert status.cpu().tolist()[0] == 0
    assert n_evictions >= 3
