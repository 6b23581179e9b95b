"""kvcrush_kmeans_select (the clustering baseline of the ablation "KMeans vs KVCrush", Fig. 3) against the oracle's
exact Lloyd iterations: kept sets and kinds must be identical."""
import numpy as np
import pytest

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(B, Hq, Hkv, seqlens, budgets, iterations, seed, n_layers=1, max_rep=None, keep_initial=0, keep_recent=0,
          use_importance=False):
    import torch
    dev = torch.device("cuda:0")
    T = int(sum(seqlens))
    cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int64)
    W = (Hq + 31) // 32
    scores = np.zeros((n_layers, Hq, T), dtype=np.float32)
    sigs = np.zeros((n_layers, T, W), dtype=np.uint32)
    bi = np.zeros((n_layers, len(seqlens)), dtype=np.int32)
    br = np.zeros((n_layers, len(seqlens)), dtype=np.int32)
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            s32 = inputs.random_scores(Hq, L, seed + 17 * l + s, tie_levels=4 if (s + l) % 2 else 0)
            scores[l, :, cu[s]:cu[s + 1]] = s32
            bi[l, s], br[l, s] = budgets[s]
            sigs[l, cu[s]:cu[s + 1]] = O.signatures(s32, O.thresholds(s32, int(bi[l, s] + br[l, s])))
    kept = np.minimum(bi.astype(np.int64) + br, np.asarray(seqlens)[None, :])
    cu_kept = np.zeros(n_layers * len(seqlens) + 1, dtype=np.int32)
    cu_kept[1:] = np.cumsum(kept.reshape(-1))
    prob = B.Problem(n_layers, Hq, Hkv, 16, seqlens, device=dev)
    K = int(br.max()) if max_rep is None else max_rep
    d_scores = torch.from_numpy(scores).to(dev)
    d_sigs = torch.from_numpy(sigs.view(np.int32)).to(dev)
    d_bi, d_br = torch.from_numpy(bi).to(dev), torch.from_numpy(br).to(dev)
    d_cu = torch.from_numpy(cu_kept).to(dev)
    idx = torch.full((max(int(cu_kept[-1]), 1),), -7, dtype=torch.int32, device=dev)
    kind = torch.full((max(int(cu_kept[-1]), 1),), 9, dtype=torch.uint8, device=dev)
    n_kept = torch.full((n_layers, len(seqlens)), -1, dtype=torch.int32, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    ws = torch.empty(max(256, B.kvcrush_kmeans_workspace_size(prob, K)), dtype=torch.uint8, device=dev)
    imp = None
    if use_importance:                      # I(t) as the signature stage hands it over
        imp = torch.empty((n_layers, T), dtype=torch.float64, device=dev)
        sig_out = torch.empty((n_layers, T, W), dtype=torch.int32, device=dev)
        keep = torch.from_numpy((bi + br).astype(np.int32)).to(dev)
        ws2 = torch.empty(max(256, B.kvcrush_workspace_size(prob, B.STAGE_SIGNATURE)), dtype=torch.uint8, device=dev)
        B.kvcrush_signature(prob, d_scores, sig_out, sig_keep=keep, importance_out=imp, workspace=ws2, status=status)
    B.kvcrush_kmeans_select(prob, None if use_importance else d_scores, d_sigs, d_bi, d_br, K, iterations, d_cu, idx,
                            importance=imp, kind=kind, n_kept=n_kept, keep_initial=keep_initial, keep_recent=keep_recent,
                            workspace=ws, status=status)
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    g_idx, g_kind, g_n = idx.cpu().numpy(), kind.cpu().numpy(), n_kept.cpu().numpy()
    if st[0] != 0:
        return st
    for l in range(n_layers):
        for s, L in enumerate(seqlens):
            seg = l * len(seqlens) + s
            s32 = np.ascontiguousarray(scores[l][:, cu[s]:cu[s + 1]])
            want, want_kind = O.kmeans_select(s32, sigs[l, cu[s]:cu[s + 1]], int(bi[l, s]), int(br[l, s]), Hkv,
                                              iterations=iterations, keep_recent=keep_recent, keep_initial=keep_initial)
            lo, hi = int(cu_kept[seg]), int(cu_kept[seg + 1])
            assert g_n[l, s] == hi - lo == want.shape[0]
            np.testing.assert_array_equal(g_idx[lo:hi], want.astype(np.int32), err_msg=f"layer {l} seq {s}")
            np.testing.assert_array_equal(g_kind[lo:hi], want_kind, err_msg=f"layer {l} seq {s}")
    return st


def test_kmeans_matches_the_oracle_bit_for_bit():
    from paper_2503_00022_b200 import binding as B, build
    build.build()
    # several tiles of clusters (k > 64), ragged batch, duplicates (tie levels), two signature words, GQA importance
    _case(B, 8, 8, [200], [(20, 30)], 3, seed=1)
    _case(B, 32, 8, [333, 64, 700], [(40, 70), (10, 20), (100, 150)], 2, seed=2, n_layers=2)
    _case(B, 40, 40, [257], [(0, 33)], 4, seed=3)
    _case(B, 8, 4, [300], [(50, 100)], 0, seed=4)                      # no iteration: initial centroids only
    _case(B, 4, 4, [400], [(30, 120)], 5, seed=5)                      # 16 distinct vectors: most clusters stay empty
    _case(B, 16, 16, [150, 90], [(20, 0), (100, 50)], 2, seed=6)       # no representatives; budget covers the sequence
    _case(B, 32, 32, [500], [(60, 60)], 3, seed=7, keep_initial=4, keep_recent=16, use_importance=True)


def test_kmeans_reports_a_budget_above_the_declared_maximum_and_rejects_bad_arguments():
    import torch
    from paper_2503_00022_b200 import binding as B, build
    build.build()
    st = _case(B, 8, 8, [100], [(10, 20)], 1, seed=8, max_rep=5)
    assert st[0] == B.DEV_BUDGET and st[2] == 0 and st[3] == 20
    dev = torch.device("cuda:0")
    prob = B.Problem(1, 8, 8, 16, [40000], device=dev)                 # longer than the baseline supports
    t = torch.zeros(8, dtype=torch.int32, device=dev)
    with pytest.raises(B.KvcrushError) as e:
        B.kvcrush_kmeans_select(prob, t, t, t, t, 4, 1, t, t, workspace=t, status=t)
    assert e.value.code == B.ERR_UNSUPPORTED
    prob = B.Problem(1, 8, 8, 16, [100], device=dev)
    with pytest.raises(B.KvcrushError) as e:
        B.kvcrush_kmeans_select(prob, t, t, t, t, 4, 1, t, t, workspace=t, status=t)     # workspace too small
    assert e.value.code == B.ERR_WORKSPACE
