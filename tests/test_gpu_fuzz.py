"""Seeded random sweeps over shapes, budgets, anchors and tie densities: the selection stages must stay
bit-exact against the oracle, the tensor-core scores must stay within tolerance of the oracle (and close to
the CUDA-core path) whatever the mix of sequence lengths."""
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


def _random_selection_cases(B, seed, n_cases, lengths, max_seqs):
    import torch
    dev = torch.device("cuda:0")
    g = np.random.Generator(np.random.Philox(seed))
    for case in range(n_cases):
        Hkv = int(g.choice([1, 2, 3, 8, 16]))
        Hq = Hkv * int(g.choice([1, 2, 4, 8]))
        if Hq > 128:
            Hq = Hkv
        n_seqs = int(g.integers(1, max_seqs + 1))
        seqlens = [int(g.choice(lengths)) for _ in range(n_seqs)]
        n_layers = int(g.integers(1, 3))
        ties = int(g.choice([0, 0, 2, 5]))
        mode = int(g.integers(0, 3))
        keep_recent = int(g.choice([0, 0, 3, 40]))
        keep_initial = int(g.choice([0, 0, 4, 33]))
        b_imp = np.asarray([int(g.integers(0, L + 1)) for L in seqlens], dtype=np.int32)
        b_rep = np.asarray([int(g.integers(0, max(1, L - bi + 1))) for L, bi in zip(seqlens, b_imp)], dtype=np.int32)
        if case % 7 == 0:
            b_rep[:] = 1                                     # one huge bucket per sequence
        T = int(sum(seqlens))
        cu = np.concatenate([[0], np.cumsum(seqlens)])
        scores = np.zeros((n_layers, Hq, T), dtype=np.float32)
        for l in range(n_layers):
            for s, L in enumerate(seqlens):
                scores[l, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, 1000 * case + 10 * l + s, tie_levels=ties)
        explicit = inputs.random_anchor_bits(Hq, 500 + case)
        prob = B.Problem(n_layers, Hq, Hkv, 16, seqlens, device=dev)
        cp = B.CompressionPass(prob, b_imp[None], b_rep[None], anchor_mode=mode,
                               anchor_bits=explicit if mode == B.ANCHOR_EXPLICIT else None, keep_recent=keep_recent,
                               keep_initial=keep_initial)
        ds = torch.from_numpy(scores).to(dev)
        cp.signature(ds)
        cp.select(ds)
        torch.cuda.synchronize()
        cp.check_status()
        sigs = cp.sigs.cpu().numpy().view(np.uint32)
        for l in range(n_layers):
            for s, L in enumerate(seqlens):
                s32 = np.ascontiguousarray(scores[l][:, cu[s]:cu[s + 1]])
                sig = O.signatures(s32, O.thresholds(s32, int(b_imp[s] + b_rep[s])))
                ctx = (case, Hq, Hkv, seqlens, b_imp.tolist(), b_rep.tolist(), ties, mode, keep_recent, keep_initial, l, s)
                assert np.array_equal(sigs[l, cu[s]:cu[s + 1]], sig), ctx
                idx, kind = O.select(s32, sig, int(b_imp[s]), int(b_rep[s]), Hkv, mode, explicit, keep_recent=keep_recent,
                                     keep_initial=keep_initial)
                assert np.array_equal(cp.kept(l, s), idx.astype(np.int32)), ctx
                seg = l * n_seqs + s
                lo, hi = int(cp.cu_kept_host[seg]), int(cp.cu_kept_host[seg + 1])
                assert np.array_equal(cp.kind[lo:hi].cpu().numpy(), kind), ctx
                assert int(cp.n_kept[l, s]) == hi - lo, ctx


def test_random_selection_problems_are_bit_exact(B):
    _random_selection_cases(B, 2024, 36, [1, 2, 31, 32, 33, 64, 100, 257, 1000, 2100], 4)


def test_random_selection_problems_with_long_segments_are_bit_exact(B):
    # few long segments beside very short ones: several keys per thread in every sweep, buckets of all sizes
    _random_selection_cases(B, 777, 20, [1, 40, 1024, 1025, 1500, 2100, 3000, 5000, 9000], 3)


def test_random_score_problems_match_oracle_and_cuda_core_path(B):
    import torch
    dev = torch.device("cuda:0")
    g = np.random.Generator(np.random.Philox(4048))
    for case in range(14):
        D = int(g.choice([64, 128, 96, 80, 32, 128]))
        Hkv = int(g.choice([1, 2, 4]))
        Hq = Hkv * int(g.choice([1, 2, 4]))
        n_seqs = int(g.integers(1, 6))
        seqlens = tuple(int(g.choice([1, 5, 127, 128, 129, 200, 256, 300, 511, 640, 900])) for _ in range(n_seqs))
        causal = bool(g.integers(0, 4) > 0)
        window = int(g.choice([0, 0, 17, 130]))
        n_layers = int(g.integers(1, 3))
        qk = inputs.FP16 if case % 3 == 2 else inputs.BF16
        w = inputs.Workload(f"fz{case}", n_layers, Hq, Hkv, D, seqlens, qk, inputs.BF16, 0.25,
                            base_seed=7000 + case, causal=causal)
        lis, q, k, _, _ = TL.stack_layers(w, range(n_layers), with_cache=False)
        prob = B.Problem(n_layers, Hq, Hkv, D, seqlens, causal=causal, device=dev, query_window=window)
        dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
        ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
        status = torch.zeros(4, dtype=torch.int32, device=dev)
        out = {}
        for name, impl in (("tensor", B.SCORE_TENSOR), ("simt", B.SCORE_SIMT)):
            sc = torch.full((n_layers, Hq, w.total_tokens), -1.0, dtype=torch.float32, device=dev)
            B.kvcrush_score(prob, dq, dk, sc, impl=impl, workspace=ws, status=status)
            torch.cuda.synchronize()
            assert status.cpu().tolist()[0] == 0
            out[name] = sc.cpu().numpy()
        ctx = (case, D, Hq, Hkv, seqlens, causal, window, qk)
        np.testing.assert_allclose(out["tensor"], out["simt"], rtol=3e-4, atol=2e-6, err_msg=str(ctx))
        cu = w.cu_seqlens
        for l, li in enumerate(lis):
            for s, L in enumerate(seqlens):
                a, b = int(cu[s]), int(cu[s + 1])
                j0 = max(0, L - window) if window else 0
                c, _ = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), causal, rows=(j0, L))
                assert TL.within_score_tolerance(out["tensor"][l][:, a:b], c).all(), ctx


def test_large_logits_stay_within_tolerance(B):
    """Logits of +-100 and more (a softmax scale 8x the usual): rows are dominated by one or two keys, the row
    maximum moves a lot between tiles, most exponentials underflow."""
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload("big", 1, 4, 2, 128, (777, 130), inputs.BF16, inputs.BF16, 0.25, base_seed=99)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    scale = 8.0 / np.sqrt(128.0)
    prob = B.Problem(1, 4, 2, 128, w.seqlens, softmax_scale=scale, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    cu = w.cu_seqlens
    for impl in (B.SCORE_TENSOR, B.SCORE_SIMT):
        sc = torch.empty((1, 4, w.total_tokens), dtype=torch.float32, device=dev)
        B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev), sc,
                        impl=impl, workspace=ws, status=status)
        torch.cuda.synchronize()
        g = sc.cpu().numpy()
        assert np.isfinite(g).all()
        for s_, L in enumerate(w.seqlens):
            a, b = int(cu[s_]), int(cu[s_ + 1])
            c, _ = O.scores(inputs.widen(lis[0].q[a:b], w.qk_dtype), inputs.widen(lis[0].k[a:b], w.qk_dtype), True, scale=scale)
            ok = TL.within_score_tolerance(g[0][:, a:b], c)
            assert ok.all(), (impl, s_, np.argwhere(~ok)[:4], g[0][:, a:b][~ok][:4], c[~ok][:4])


@pytest.mark.parametrize("D", [96, 80, 8])
def test_head_dims_between_the_kernel_widths(B, D):
    """head_dim 96 (Phi-3-mini, one of the paper's models) and other multiples of 8 run in the next wider tensor-core
    kernel with the missing channels read as zeros."""
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload(f"d{D}", 1, 4, 2, D, (700, 129), inputs.BF16, inputs.BF16, 0.25, base_seed=300 + D)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    prob = B.Problem(1, 4, 2, D, w.seqlens, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    sc = torch.empty((1, 4, w.total_tokens), dtype=torch.float32, device=dev)
    B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev), sc,
                    impl=B.SCORE_TENSOR, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    got = sc.cpu().numpy()
    cu = w.cu_seqlens
    for s_, L in enumerate(w.seqlens):
        a, b = int(cu[s_]), int(cu[s_ + 1])
        c, _ = O.scores(inputs.widen(lis[0].q[a:b], w.qk_dtype), inputs.widen(lis[0].k[a:b], w.qk_dtype), True)
        assert TL.within_score_tolerance(got[0][:, a:b], c).all(), (D, s_)


def test_logit_jumps_of_hundreds_between_tiles(B):
    """Keys whose norm jumps by 60x after the first tiles: the row maximum moves by hundreds (log2 domain) between
    tiles, and every running sum is rescaled by factors far below the smallest normal number."""
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload("jump", 1, 2, 2, 128, (1500,), inputs.BF16, inputs.BF16, 0.25, base_seed=123)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    kf = inputs.widen(k[0], w.qk_dtype).astype(np.float32)
    kf[200:] *= 60.0
    kf[700:] *= 4.0
    kf[1300:] *= 0.001
    k2 = inputs.to_storage(kf, w.qk_dtype)[None]
    prob = B.Problem(1, 2, 2, 128, w.seqlens, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    c, _ = O.scores(inputs.widen(q[0], w.qk_dtype), inputs.widen(k2[0], w.qk_dtype), True)
    for impl in (B.SCORE_TENSOR, B.SCORE_SIMT):
        sc = torch.empty((1, 2, 1500), dtype=torch.float32, device=dev)
        B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k2, w.qk_dtype, dev), sc,
                        impl=impl, workspace=ws, status=status)
        torch.cuda.synchronize()
        g = sc.cpu().numpy()[0]
        assert np.isfinite(g).all()
        ok = TL.within_score_tolerance(g, c)
        assert ok.all(), (impl, np.argwhere(~ok)[:4], g[~ok][:4], c[~ok][:4])


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_key_norm_profiles(B, seed):
    """Key norms that change by random factors between 1e-2 and 1e2 from one block of 64 tokens to the next, queries
    likewise: row maxima move up and down by arbitrary amounts from tile to tile."""
    import torch
    dev = torch.device("cuda:0")
    g = np.random.Generator(np.random.Philox(900 + seed))
    L = int(g.choice([1111, 1664, 2049]))
    w = inputs.Workload("norms", 1, 4, 2, 128, (L,), inputs.BF16, inputs.BF16, 0.25, base_seed=500 + seed)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    qf = inputs.widen(q[0], w.qk_dtype).astype(np.float32)
    kf = inputs.widen(k[0], w.qk_dtype).astype(np.float32)
    for a in range(0, L, 64):
        kf[a:a + 64] *= np.float32(10.0 ** g.uniform(-2, 2))
        qf[a:a + 64] *= np.float32(10.0 ** g.uniform(-1, 1))
    q2, k2 = inputs.to_storage(qf, w.qk_dtype)[None], inputs.to_storage(kf, w.qk_dtype)[None]
    prob = B.Problem(1, 4, 2, 128, w.seqlens, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    c, lse = O.scores(inputs.widen(q2[0], w.qk_dtype), inputs.widen(k2[0], w.qk_dtype), True)
    sc = torch.empty((1, 4, L), dtype=torch.float32, device=dev)
    lo = torch.empty_like(sc)
    B.kvcrush_score(prob, TL.torch_storage(q2, w.qk_dtype, dev), TL.torch_storage(k2, w.qk_dtype, dev), sc, lse_out=lo,
                    impl=B.SCORE_TENSOR, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    gl = lo.cpu().numpy()[0]
    np.testing.assert_allclose(gl, lse, rtol=2e-6, atol=1e-3)
    ok = TL.within_score_tolerance(sc.cpu().numpy()[0], c)
    assert ok.all(), (seed, np.argwhere(~ok)[:4])
