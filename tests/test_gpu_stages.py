"""GPU parity, stage by stage, through the C ABI: signature, selection and compaction are
bit-exact when fed the oracle's float32 scores; scores agree within 1e-5 + 2e-3*|oracle|."""
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


# ---------------------------------------------------------------------------------------------
# signature + select on oracle scores
# ---------------------------------------------------------------------------------------------

def _select_case(B, Hq, Hkv, seqlens, budgets, n_layers, ties, mode, seed, sig_keep=None, share_importance=True):
    import torch
    dev = _dev()
    S, T = len(seqlens), int(sum(seqlens))
    cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int64)
    b_imp = np.asarray([b[0] for b in budgets], dtype=np.int32)
    b_rep = np.asarray([b[1] for b in budgets], dtype=np.int32)
    scores = np.zeros((n_layers, Hq, T), dtype=np.float32)
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            scores[l, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, seed + 17 * l + s, tie_levels=ties)
    explicit = inputs.random_anchor_bits(Hq, seed + 5)
    w = inputs.Workload("t", n_layers, Hq, Hkv, 16, tuple(seqlens), inputs.FP32, inputs.FP32, 0.25)
    prob = B.Problem(n_layers, Hq, Hkv, 16, seqlens, device=dev)
    # share_importance: the signature stage writes the token importance and the selection stage takes it over;
    # without it the selection stage makes its own pass over the scores
    cp = B.CompressionPass(prob, b_imp[None, :], b_rep[None, :], sig_keep=sig_keep, anchor_mode=mode,
                           anchor_bits=explicit if mode == B.ANCHOR_EXPLICIT else None,
                           share_importance=share_importance)
    dscores = torch.from_numpy(scores).to(dev)
    for rep in range(2):                      # twice: results must not depend on leftover scratch
        cp.signature(dscores)
        cp.select(dscores)
        torch.cuda.synchronize()
        cp.check_status()
        sigs = cp.sigs.cpu().numpy().view(np.uint32)
        theta = cp.theta.cpu().numpy()
        np.testing.assert_array_equal(cp.n_kept.cpu().numpy(),        # the optional per-segment count output
                                      np.tile(np.minimum(b_imp + b_rep, np.asarray(seqlens)), (n_layers, 1)))
        for l in range(n_layers):
            ref = TL.oracle_select_layer(w, scores[l], b_imp, b_rep,
                                         None if sig_keep is None else np.asarray(sig_keep).reshape(-1),
                                         mode, explicit)
            for s in range(S):
                np.testing.assert_array_equal(theta[l, s], ref[s]["theta"])
                np.testing.assert_array_equal(sigs[l, cu[s]:cu[s + 1]], ref[s]["sig"])
                np.testing.assert_array_equal(cp.kept(l, s), ref[s]["idx"].astype(np.int32))
                seg = l * S + s
                kind = cp.kind[int(cp.cu_kept_host[seg]):int(cp.cu_kept_host[seg + 1])].cpu().numpy()
                np.testing.assert_array_equal(kind, ref[s]["kind"])


@pytest.mark.parametrize("Hq,Hkv,seqlens,budgets,ties,mode", [
    (8, 8, [512], [(64, 64)], 0, 0),
    (32, 32, [4096], [(512, 512)], 0, 0),
    (32, 8, [1000, 37, 2049], [(100, 150), (5, 4), (300, 212)], 0, 0),
    (32, 8, [1000, 333], [(100, 150), (40, 43)], 4, 0),            # heavy ties everywhere
    (40, 10, [777, 1025], [(64, 32), (100, 101)], 2, 1),           # two signature words, MEAN anchor
    (128, 16, [600], [(50, 70)], 0, 2),                            # four words, explicit (random) anchor
    (4, 1, [300, 300], [(0, 30), (30, 0)], 3, 0),                  # pure KVCrush / pure H2O
    (16, 16, [100, 1, 64], [(60, 60), (1, 0), (3, 1)], 0, 1),      # budget >= length keeps all; L = 1
    (32, 32, [5000], [(10, 1)], 0, 0),                             # one huge bucket
    (32, 32, [2500], [(20, 2)], 2, 1),
])
def test_signature_and_select_bit_exact_on_oracle_scores(B, Hq, Hkv, seqlens, budgets, ties, mode):
    _select_case(B, Hq, Hkv, seqlens, budgets, 2, ties, mode, seed=100 + Hq + len(seqlens))


def test_select_long_sequence_32k(B):
    _select_case(B, 32, 8, [32768], [(3277, 3277)], 1, 0, 0, seed=9)
    _select_case(B, 32, 8, [32768], [(3277, 3277)], 1, 0, 0, seed=9, share_importance=False)


@pytest.mark.parametrize("Hq,Hkv,seqlens,budgets,ties,mode", [
    (32, 8, [1000, 37, 2049], [(100, 150), (5, 4), (300, 212)], 0, 0),
    (32, 8, [1000, 333], [(100, 150), (40, 43)], 4, 0),
    (40, 10, [777, 1025], [(64, 32), (100, 101)], 2, 1),
])
def test_select_computes_the_importance_itself_when_none_is_handed_over(B, Hq, Hkv, seqlens, budgets, ties, mode):
    _select_case(B, Hq, Hkv, seqlens, budgets, 2, ties, mode, seed=300 + Hq, share_importance=False)


def test_signature_thresholds_for_rows_beyond_the_register_kernel(B):
    """Rows longer than 32768 tokens take the streaming threshold kernel."""
    _select_case(B, 4, 2, [40000, 70], [(500, 300), (7, 9)], 1, 0, 0, seed=17)
    _select_case(B, 4, 2, [33000], [(100, 50)], 1, 3, 0, seed=18)


def test_signature_rank_other_than_budget_and_explicit_theta(B):
    import torch
    dev = _dev()
    _select_case(B, 16, 4, [400, 250], [(30, 30), (20, 21)], 1, 0, 0, seed=3, sig_keep=[[30, 20]])
    # explicit thresholds (the input form of Algorithm 1)
    Hq, L = 24, 333
    s = inputs.random_scores(Hq, L, 12)
    theta = np.linspace(0.05, 3.0, Hq).astype(np.float32)
    prob = B.Problem(1, Hq, Hq, 16, [L], device=dev)
    sigs = torch.empty((1, L, 1), dtype=torch.int32, device=dev)
    tout = torch.empty((1, 1, Hq), dtype=torch.float32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_signature(prob, torch.from_numpy(s[None]).to(dev), sigs, theta_in=torch.from_numpy(theta).to(dev),
                        theta_out=tout, status=status)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(sigs.cpu().numpy().view(np.uint32)[0], O.signatures(s, theta))
    np.testing.assert_array_equal(tout.cpu().numpy().reshape(-1), theta)


# ---------------------------------------------------------------------------------------------
# compaction
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,D,Hkv,layout", [
    (inputs.FP16, 128, 8, "thd"), (inputs.BF16, 128, 4, "htd"), (inputs.FP32, 64, 8, "thd"), (inputs.BF16, 64, 3, "thd"),
])
def test_compact_bytes_equal_oracle(B, dtype, D, Hkv, layout):
    import torch
    dev = _dev()
    seqlens, n_layers = [300, 45, 1000], 3
    w = inputs.Workload("c", n_layers, Hkv, Hkv, D, tuple(seqlens), dtype, dtype, 0.25, base_seed=77)
    lis, _, _, kc, vc = TL.stack_layers(w, range(n_layers))
    g = np.random.Generator(np.random.Philox(5))
    budgets = np.asarray([[g.integers(1, L + 1) for L in seqlens] for _ in range(n_layers)], dtype=np.int32)
    prob = B.Problem(n_layers, Hkv, Hkv, D, seqlens, device=dev)
    tdt = {inputs.FP16: torch.float16, inputs.BF16: torch.bfloat16, inputs.FP32: torch.float32}[dtype]
    cp = B.CompressionPass(prob, budgets, np.zeros_like(budgets), cache_dtype=tdt)
    cu = w.cu_seqlens
    idx_host, ref_k, ref_v = [], [], []
    for l in range(n_layers):
        rk, rv = [], []
        for s, L in enumerate(seqlens):
            idx = np.sort(g.choice(L, size=int(budgets[l, s]), replace=False))
            idx_host.append(idx)
            rk.append(O.compact(kc[l, cu[s]:cu[s + 1]], idx))
            rv.append(O.compact(vc[l, cu[s]:cu[s + 1]], idx))
        ref_k.append(np.concatenate(rk))
        ref_v.append(np.concatenate(rv))
    cp.idx.copy_(torch.from_numpy(np.concatenate(idx_host).astype(np.int32)).to(dev))
    dk, dv = TL.torch_storage(kc, dtype, dev), TL.torch_storage(vc, dtype, dev)
    if layout == "htd":      # cache stored [layer, head, token, D]; the ABI sees it through strides
        dk = dk.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        dv = dv.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    cp.k_out.fill_(0)
    cp.v_out.fill_(0)
    cp.compact(dk, dv)
    torch.cuda.synchronize()
    for l in range(n_layers):
        n = ref_k[l].shape[0]
        got_k = cp.k_out[l, :n].contiguous().view(torch.uint8).cpu().numpy()
        got_v = cp.v_out[l, :n].contiguous().view(torch.uint8).cpu().numpy()
        assert got_k.tobytes() == ref_k[l].tobytes()
        assert got_v.tobytes() == ref_v[l].tobytes()
        rest = cp.k_out[l, n:].contiguous().view(torch.uint8)
        assert int(rest.max()) == 0 if rest.numel() else True       # nothing written past the kept rows


# ---------------------------------------------------------------------------------------------
# scores
# ---------------------------------------------------------------------------------------------

def _score_case(B, w, impl, n_layers=None):
    import torch
    dev = _dev()
    layers = range(w.n_layers if n_layers is None else n_layers)
    lis, q, k, _, _ = TL.stack_layers(w, layers, with_cache=False)
    prob = B.Problem(len(lis), w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, causal=w.causal, device=dev)
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    T = w.total_tokens
    scores = torch.full((len(lis), w.n_q_heads, T), -1.0, dtype=torch.float32, device=dev)
    lse = torch.empty_like(scores)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_score(prob, dq, dk, scores, lse_out=lse, impl=impl, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0, status.cpu().tolist()
    g, gl = scores.cpu().numpy(), lse.cpu().numpy()
    oracle_c, oracle_lse = [], []
    for i, li in enumerate(lis):
        c, ol = TL.oracle_scores_layer(w, li)
        ok = TL.within_score_tolerance(g[i], c)
        assert ok.all(), (w.name, i, np.argwhere(~ok)[:5], g[i][~ok][:5], c[~ok][:5])
        np.testing.assert_allclose(gl[i], ol, rtol=0, atol=2e-4)
        oracle_c.append(c)
        oracle_lse.append(ol)
    # the row log-sum-exp as a prefill kernel would hand it over - here the ORACLE's, rounded to float32, so that
    # nothing of the library's first sweep is involved: the second sweep alone must reproduce the oracle's column sums
    lse_o = torch.from_numpy(np.stack(oracle_lse).astype(np.float32)).to(dev)
    scores3 = torch.full_like(scores, -1.0)
    B.kvcrush_score(prob, dq, dk, scores3, lse_in=lse_o, impl=impl, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    g3 = scores3.cpu().numpy()
    for i, c in enumerate(oracle_c):
        ok = TL.within_score_tolerance(g3[i], c)
        assert ok.all(), (w.name, "oracle lse", i, np.argwhere(~ok)[:5], g3[i][~ok][:5], c[~ok][:5])
    # supplying the row log-sum-exp skips the first sweep and gives the same scores
    scores2 = torch.empty_like(scores)
    B.kvcrush_score(prob, dq, dk, scores2, lse_in=lse, impl=impl, workspace=ws, status=status)
    torch.cuda.synchronize()
    np.testing.assert_allclose(scores2.cpu().numpy(), g, rtol=1e-4, atol=1e-6)
    # normalize = the paper's 1/S
    B.kvcrush_score(prob, dq, dk, scores2, normalize=True, impl=impl, workspace=ws, status=status)
    torch.cuda.synchronize()
    cu = w.cu_seqlens
    n2 = scores2.cpu().numpy()
    for s, L in enumerate(w.seqlens):
        np.testing.assert_allclose(n2[:, :, cu[s]:cu[s + 1]] * L, g[:, :, cu[s]:cu[s + 1]], rtol=1e-5, atol=1e-7)
    return g


SIMT_CASES = [
    inputs.Workload("simt_cfg1", 1, 8, 8, 64, (512,), inputs.FP32, inputs.FP32, 0.25, base_seed=1100),
    inputs.Workload("simt_ragged_gqa", 2, 8, 2, 32, (130, 1, 257), inputs.BF16, inputs.BF16, 0.25, base_seed=21),
    inputs.Workload("simt_noncausal", 1, 4, 4, 128, (200, 96), inputs.BF16, inputs.BF16, 0.25, base_seed=22, causal=False),
]


@pytest.mark.parametrize("w", SIMT_CASES, ids=lambda w: w.name)
def test_score_simt_matches_oracle(B, w):
    _score_case(B, w, B.SCORE_SIMT)


TENSOR_CASES = [
    inputs.Workload("tc_one_tile", 1, 2, 2, 128, (128,), inputs.BF16, inputs.BF16, 0.25, base_seed=31),
    inputs.Workload("tc_ragged_tail", 1, 4, 4, 128, (700,), inputs.BF16, inputs.BF16, 0.25, base_seed=32),
    inputs.Workload("tc_gqa_varlen", 2, 8, 2, 128, (300, 1, 129, 1000), inputs.BF16, inputs.BF16, 0.25, base_seed=33),
    inputs.Workload("tc_d64", 1, 4, 2, 64, (513, 64), inputs.BF16, inputs.BF16, 0.25, base_seed=34),
    inputs.Workload("tc_noncausal", 1, 4, 4, 128, (333, 260), inputs.BF16, inputs.BF16, 0.25, base_seed=35, causal=False),
    inputs.Workload("tc_2k", 1, 8, 8, 128, (2048,), inputs.BF16, inputs.BF16, 0.25, base_seed=36),
    # more sequences than one warp decodes at once, lengths around every tile / block boundary, an empty sequence
    inputs.Workload("tc_many_seqs", 1, 2, 1, 64, tuple([127, 128, 129, 255, 256, 257, 0, 1, 383, 384, 385, 512] * 3 + [40, 300]),
                    inputs.BF16, inputs.BF16, 0.25, base_seed=37),
    inputs.Workload("tc_128_heads", 1, 128, 16, 64, (260,), inputs.BF16, inputs.BF16, 0.25, base_seed=38),
]


@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_score_tensor_matches_oracle(B, w):
    g = _score_case(B, w, B.SCORE_TENSOR)
    # the CUDA-core kernels see the same inputs: the two device paths agree far inside the tolerance
    import torch
    dev = _dev()
    lis, q, k, _, _ = TL.stack_layers(w, range(w.n_layers), with_cache=False)
    prob = B.Problem(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, causal=w.causal, device=dev)
    scores = torch.empty((w.n_layers, w.n_q_heads, w.total_tokens), dtype=torch.float32, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev), scores,
                    impl=B.SCORE_SIMT, workspace=ws, status=status)
    torch.cuda.synchronize()
    np.testing.assert_allclose(g, scores.cpu().numpy(), rtol=2e-4, atol=1e-6)


def test_score_tensor_rejects_fp32_and_auto_falls_back_to_cuda_cores(B):
    import torch
    dev = _dev()
    w = SIMT_CASES[0]
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    prob = B.Problem(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, device=dev)
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    scores = torch.empty((1, w.n_q_heads, w.total_tokens), dtype=torch.float32, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(B.KvcrushError) as e:
        B.kvcrush_score(prob, dq, dk, scores, impl=B.SCORE_TENSOR, workspace=ws, status=status)
    assert e.value.code == B.ERR_UNSUPPORTED
    B.kvcrush_score(prob, dq, dk, scores, impl=B.SCORE_AUTO, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert torch.isfinite(scores).all()


@pytest.mark.parametrize("impl_name", ["SCORE_TENSOR", "SCORE_SIMT"])
def test_score_head_major_layout_and_explicit_scale(B, impl_name):
    """Q/K stored [layer, head, token, D] (reached through strides) and a caller-chosen softmax scale."""
    import torch
    dev = _dev()
    impl = getattr(B, impl_name)
    w = inputs.Workload("hm", 2, 4, 2, 128, (391, 130), inputs.BF16, inputs.BF16, 0.25, base_seed=41)
    lis, q, k, _, _ = TL.stack_layers(w, range(2), with_cache=False)
    scale = 0.05
    prob = B.Problem(2, 4, 2, 128, w.seqlens, causal=True, softmax_scale=scale, device=dev)
    dq = TL.torch_storage(q, w.qk_dtype, dev).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    dk = TL.torch_storage(k, w.qk_dtype, dev).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert dq.stride(1) == 128 and dq.stride(2) == 128 * w.total_tokens
    scores = torch.empty((2, 4, w.total_tokens), dtype=torch.float32, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.kvcrush_score(prob, dq, dk, scores, impl=impl, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    g = scores.cpu().numpy()
    cu = w.cu_seqlens
    for l, li in enumerate(lis):
        for s_, L in enumerate(w.seqlens):
            a, b = int(cu[s_]), int(cu[s_ + 1])
            c, _ = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), True, scale=scale)
            assert TL.within_score_tolerance(g[l][:, a:b], c).all()


def test_score_leaves_at_once_when_status_already_flags_an_error(B):
    """The tensor-core kernels read the status word first: a launch that follows a reported device error does
    no work (outputs untouched) and keeps the first error's record."""
    import torch
    dev = _dev()
    w = TENSOR_CASES[1]
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    prob = B.Problem(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, device=dev)
    scores = torch.full((1, w.n_q_heads, w.total_tokens), -5.0, dtype=torch.float32, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.tensor([B.DEV_TIMEOUT, 2, 17, 0], dtype=torch.int32, device=dev)
    B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev), scores,
                    impl=B.SCORE_TENSOR, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [B.DEV_TIMEOUT, 2, 17, 0]
    assert bool((scores == -5.0).all())
    status.zero_()                                           # and the same call works once the word is cleared
    B.kvcrush_score(prob, TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev), scores,
                    impl=B.SCORE_TENSOR, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0 and bool((scores >= 0).all())


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable(B):
    """Every barrier wait of the tensor-core kernels is bounded.  Here one is made to run out, on the smallest problem
    there is (one work item, one thread block): through the library's diagnostic entry point (exported, not part of
    the public header) the producer warp fetches its work item and then stops before announcing it and before issuing
    any copy, and the kernels run in their instantiation with a short poll limit.  Nothing is in flight, so the
    consumers' first waits expire, the block flags the status word, frees its tensor memory and the kernel returns
    normally; the second sweep, enqueued by the same call, finds the status word set and leaves at once.  The outputs
    stay untouched, and the same problem goes through the public entry point once the word is cleared."""
    import ctypes
    import torch
    dev = _dev()
    lib = B.lib()
    fn = lib.kvcrush_diag_score
    vp, i32 = ctypes.c_void_p, ctypes.c_int
    fn.restype = i32
    fn.argtypes = [ctypes.POINTER(B.ProblemStruct), ctypes.POINTER(B.TensorStruct), ctypes.POINTER(B.TensorStruct),
                   vp, vp, vp, i32, i32, vp, ctypes.c_size_t, vp, vp, i32, i32]
    w = inputs.Workload("one_item", 1, 1, 1, 128, (128,), inputs.BF16, inputs.BF16, 0.25, base_seed=55)
    lis, q, k, _, _ = TL.stack_layers(w, range(1), with_cache=False)
    prob = B.Problem(1, 1, 1, 128, w.seqlens, device=dev)
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    qs, ks = B.tensor_struct(dq), B.tensor_struct(dk)
    scores = torch.full((1, 1, 128), -5.0, dtype=torch.float32, device=dev)
    lse = torch.full((1, 1, 128), -7.0, dtype=torch.float32, device=dev)
    ws = torch.empty(B.kvcrush_workspace_size(prob, B.STAGE_SCORE), dtype=torch.uint8, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    stream = int(torch.cuda.current_stream().cuda_stream)
    rc = fn(prob.ref, ctypes.byref(qs), ctypes.byref(ks), None, scores.data_ptr(), lse.data_ptr(), 0, B.SCORE_TENSOR,
            ws.data_ptr(), ws.numel(), status.data_ptr(), stream, 1, 1)
    assert rc == B.OK
    torch.cuda.synchronize()                                 # the kernels came back by themselves
    st = status.cpu().tolist()
    assert st[0] == B.DEV_TIMEOUT and st[1] == 1 and st[2] == 0, st          # kernel id 1: the row sweep; block 0
    assert bool((scores == -5.0).all()) and bool((lse == -7.0).all())
    # the public entry point gives the oracle's scores on the same context once the word is cleared
    status.zero_()
    scores.fill_(-5.0)
    B.kvcrush_score(prob, dq, dk, scores, lse_out=lse, impl=B.SCORE_TENSOR, workspace=ws, status=status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == 0
    c, ol = TL.oracle_scores_layer(w, lis[0])
    assert TL.within_score_tolerance(scores.cpu().numpy()[0], c).all()
    np.testing.assert_allclose(lse.cpu().numpy()[0], ol, rtol=0, atol=2e-4)


def test_pass_replays_from_a_cuda_graph(B):
    """The four stages enqueue kernels and one memset only, so a pass can be recorded once and replayed on new
    contents of the same tensors; the replayed result equals a direct run."""
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload("graph", 2, 8, 2, 128, (600, 259), inputs.BF16, inputs.FP16, 0.25, base_seed=81)
    lis, q, k, kc, vc = TL.stack_layers(w, range(2))
    prob = B.Problem(2, 8, 2, 128, w.seqlens, device=dev)
    b_imp, b_rep = w.budgets()
    dq, dk = TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev)
    dkc, dvc = TL.torch_storage(kc, w.cache_dtype, dev), TL.torch_storage(vc, w.cache_dtype, dev)
    direct = B.CompressionPass(prob, b_imp[None], b_rep[None], cache_dtype=torch.float16)
    direct.run(dq, dk, dkc, dvc)
    torch.cuda.synchronize()
    want = (direct.idx.clone(), direct.k_out.clone(), direct.scores.clone())
    cp = B.CompressionPass(prob, b_imp[None], b_rep[None], cache_dtype=torch.float16)
    zq, zk = torch.zeros_like(dq), torch.zeros_like(dk)
    cp.capture(zq, zk, dkc, dvc)                     # recorded on other contents
    zq.copy_(dq)
    zk.copy_(dk)
    for _ in range(2):
        cp.replay()
    torch.cuda.synchronize()
    cp.check_status()
    assert torch.equal(cp.idx, want[0]) and torch.equal(cp.k_out, want[1]) and torch.equal(cp.scores, want[2])
