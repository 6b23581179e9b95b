"""GPU parity of page- and chunk-granular KVCrush (Sec. 4.3.4: chunks of 8 tokens; Sec. 4.3.5: pages of 32 tokens):
kept pages and kinds bit-exact against the oracle, the paged reduced cache byte-equal."""
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


def _run_pages(B, scores, Hkv, seqlens, P, b_imp, b_rep, mode=0, explicit=None, keep=(0, 0)):
    import torch
    dev = torch.device("cuda:0")
    n_layers, Hq, _ = scores.shape
    prob = B.Problem(n_layers, Hq, Hkv, 16, seqlens, device=dev)
    cp = B.CompressionPass(prob, b_imp, b_rep, anchor_mode=mode,
                           anchor_bits=explicit if mode == B.ANCHOR_EXPLICIT else None, page_size=P,
                           keep_initial=keep[0], keep_recent=keep[1])
    ds = torch.from_numpy(scores).to(dev)
    cp.signature(ds)
    cp.select(ds)
    torch.cuda.synchronize()
    cp.check_status()
    pages = (np.asarray(seqlens, dtype=np.int64) + P - 1) // P
    want = np.minimum(np.broadcast_to(np.asarray(b_imp, dtype=np.int64) + np.asarray(b_rep), (n_layers, len(seqlens))), pages[None])
    np.testing.assert_array_equal(cp.n_kept.cpu().numpy(), want)         # the optional per-segment count output
    return cp


def _check_pages(cp, scores, Hkv, seqlens, P, b_imp, b_rep, mode=0, explicit=None, ctx=None, keep=(0, 0)):
    n_layers = scores.shape[0]
    cu = np.concatenate([[0], np.cumsum(seqlens)])
    b_imp = np.broadcast_to(np.asarray(b_imp), (n_layers, len(seqlens)))
    b_rep = np.broadcast_to(np.asarray(b_rep), (n_layers, len(seqlens)))
    for l in range(n_layers):
        for s in range(len(seqlens)):
            s32 = np.ascontiguousarray(scores[l][:, cu[s]:cu[s + 1]])
            bi, br = int(b_imp[l, s]), int(b_rep[l, s])
            sig = O.signatures(s32, O.thresholds(s32, (bi + br) * P))
            idx, kind = O.select_pages(s32, sig, P, bi, br, Hkv, mode, explicit, keep_initial=keep[0], keep_recent=keep[1])
            np.testing.assert_array_equal(cp.kept(l, s), idx.astype(np.int32), err_msg=str((ctx, l, s)))
            seg = l * len(seqlens) + s
            lo, hi = int(cp.cu_kept_host[seg]), int(cp.cu_kept_host[seg + 1])
            np.testing.assert_array_equal(cp.kind[lo:hi].cpu().numpy(), kind, err_msg=str((ctx, l, s)))


def _scores(n_layers, Hq, seqlens, seed, ties=0):
    T = int(sum(seqlens))
    cu = np.concatenate([[0], np.cumsum(seqlens)])
    out = np.zeros((n_layers, Hq, T), dtype=np.float32)
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            out[l, :, cu[s]:cu[s + 1]] = inputs.random_scores(Hq, L, seed + 10 * l + s, tie_levels=ties)
    return out


@pytest.mark.parametrize("P", [8, 32])
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_pages_match_oracle(B, P, mode):
    seqlens, Hq, Hkv = [1000, 37, 256, 2049], 32, 8
    scores = _scores(2, Hq, seqlens, 400 + P, ties=3 * mode)
    n_pages = [(L + P - 1) // P for L in seqlens]
    b_imp = np.asarray([max(1, n // 8) for n in n_pages], dtype=np.int32)[None]
    b_rep = np.asarray([max(1, n // 6) for n in n_pages], dtype=np.int32)[None]
    explicit = inputs.random_anchor_bits(Hq, 31)
    cp = _run_pages(B, scores, Hkv, seqlens, P, b_imp, b_rep, mode, explicit)
    _check_pages(cp, scores, Hkv, seqlens, P, b_imp, b_rep, mode, explicit)


def test_page_size_one_equals_token_level_kernel(B):
    import torch
    seqlens, Hq, Hkv = [700, 129], 40, 8
    scores = _scores(1, Hq, seqlens, 77, ties=2)
    b_imp = np.asarray([[60, 10]], dtype=np.int32)
    b_rep = np.asarray([[90, 20]], dtype=np.int32)
    cp = _run_pages(B, scores, Hkv, seqlens, 1, b_imp, b_rep)
    dev = torch.device("cuda:0")
    prob = B.Problem(1, Hq, Hkv, 16, seqlens, device=dev)
    ct = B.CompressionPass(prob, b_imp, b_rep)
    ds = torch.from_numpy(scores).to(dev)
    ct.signature(ds)
    ct.select(ds)
    torch.cuda.synchronize()
    for s in range(2):
        np.testing.assert_array_equal(cp.kept(0, s), ct.kept(0, s))
    assert torch.equal(cp.kind, ct.kind)


def test_random_page_problems_are_bit_exact(B):
    g = np.random.Generator(np.random.Philox(909))
    for case in range(30):
        Hkv = int(g.choice([1, 2, 8]))
        Hq = Hkv * int(g.choice([1, 4, 5]))
        P = int(g.choice([1, 2, 3, 8, 16, 32]))
        if P * ((Hq + 31) // 32) > 128:
            P = 8
        n_seqs = int(g.integers(1, 4))
        seqlens = [int(g.choice([1, 5, 31, 32, 33, 64, 100, 257, 1000, 3000])) for _ in range(n_seqs)]
        n_pages = [(L + P - 1) // P for L in seqlens]
        mode = int(g.integers(0, 3))
        ties = int(g.choice([0, 0, 2, 6]))
        b_imp = np.asarray([int(g.integers(0, n + 1)) for n in n_pages], dtype=np.int32)
        b_rep = np.asarray([int(g.integers(0, max(1, n - bi + 1))) for n, bi in zip(n_pages, b_imp)], dtype=np.int32)
        if case % 6 == 0:
            b_rep[:] = 1                                   # one bucket holding every grouped page
        scores = _scores(1, Hq, seqlens, 5000 + 20 * case, ties=ties)
        explicit = inputs.random_anchor_bits(Hq, 600 + case)
        keep = (int(g.choice([0, 0, 1, 3])), int(g.choice([0, 0, 2, 5])))
        cp = _run_pages(B, scores, Hkv, seqlens, P, b_imp[None], b_rep[None], mode, explicit, keep)
        _check_pages(cp, scores, Hkv, seqlens, P, b_imp[None], b_rep[None], mode, explicit,
                     ctx=(case, Hq, Hkv, P, seqlens, b_imp.tolist(), b_rep.tolist(), mode, ties, keep), keep=keep)


def test_paged_budget_of_table1(B):
    # 672 tokens = 32 initial + 512 middle + 128 recent at page size 32: 1 + 16 + 4 pages, 4 of the middle by KVCrush
    seqlens = [4000, 2500]
    scores = _scores(2, 32, seqlens, 88)
    b_imp, b_rep = np.asarray([[17, 17]], dtype=np.int32), np.asarray([[4, 4]], dtype=np.int32)
    cp = _run_pages(B, scores, 8, seqlens, 32, b_imp, b_rep, keep=(1, 4))
    _check_pages(cp, scores, 8, seqlens, 32, b_imp, b_rep, keep=(1, 4))
    for s, L in enumerate(seqlens):
        n_pages = (L + 31) // 32
        assert {0} | set(range(n_pages - 4, n_pages)) <= set(cp.kept(0, s).tolist())


def test_widest_page_vector_and_most_pages(B):
    # 128 heads x 32 tokens = 128 words per page vector (the limit); 8192 chunks of 4 tokens (the limit)
    scores = _scores(1, 128, [700], 3)
    cp = _run_pages(B, scores, 128, [700], 32, np.asarray([[3]], dtype=np.int32), np.asarray([[5]], dtype=np.int32), 1)
    _check_pages(cp, scores, 128, [700], 32, [[3]], [[5]], 1)
    scores = _scores(1, 4, [32765], 4)
    cp = _run_pages(B, scores, 2, [32765], 4, np.asarray([[1000]], dtype=np.int32), np.asarray([[700]], dtype=np.int32))
    _check_pages(cp, scores, 2, [32765], 4, [[1000]], [[700]])


def test_paged_pass_end_to_end_with_reduced_cache(B):
    """Scores on the tensor cores -> signatures -> page selection -> paged gather (ragged last pages, zero fill)."""
    import torch
    dev = torch.device("cuda:0")
    w = inputs.Workload("paged", 2, 8, 2, 128, (900, 411), inputs.BF16, inputs.FP16, 0.25, base_seed=71)
    P = 32
    lis, q, k, kc, vc = TL.stack_layers(w, range(2))
    prob = B.Problem(2, 8, 2, 128, w.seqlens, device=dev)
    b_imp = np.asarray([[4, 2]], dtype=np.int32)
    b_rep = np.asarray([[4, 11]], dtype=np.int32)            # sequence 1: 13 pages, all kept incl. the short one
    cp = B.CompressionPass(prob, b_imp, b_rep, cache_dtype=torch.float16, page_size=P)
    cp.run(TL.torch_storage(q, w.qk_dtype, dev), TL.torch_storage(k, w.qk_dtype, dev),
           TL.torch_storage(kc, w.cache_dtype, dev), TL.torch_storage(vc, w.cache_dtype, dev))
    torch.cuda.synchronize()
    cp.check_status()
    g = cp.scores.cpu().numpy()
    cu = w.cu_seqlens
    for l, li in enumerate(lis):
        for s, L in enumerate(w.seqlens):
            a, b = int(cu[s]), int(cu[s + 1])
            s32 = np.ascontiguousarray(g[l][:, a:b])
            bi, br = int(b_imp[0, s]), int(b_rep[0, s])
            sig = O.signatures(s32, O.thresholds(s32, (bi + br) * P))
            idx, kind = O.select_pages(s32, sig, P, bi, br, 2)
            np.testing.assert_array_equal(cp.kept(l, s), idx.astype(np.int32))
            seg = l * w.n_seqs + s
            lo = (int(cp.cu_kept_host[seg]) - int(cp.cu_kept_host[l * w.n_seqs])) * P
            for name, out, cache in (("k", cp.k_out, li.k_cache), ("v", cp.v_out, li.v_cache)):
                got = out[l, lo:lo + len(idx) * P].cpu().numpy()
                want = O.compact_pages(cache[a:b], idx, P)
                assert got.tobytes() == want.tobytes(), (name, l, s)
    assert 12 in cp.kept(0, 1)                               # the short last page of sequence 1 is there
