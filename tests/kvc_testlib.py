"""Shared helpers of the tests: run the oracle per (layer, sequence) and stage tensors for the GPU."""
import numpy as np

from oracle import kvcrush_oracle as O
from paper_2503_00022_b200 import inputs

SCORE_RTOL, SCORE_ATOL = 2e-3, 1e-5      # |gpu - oracle| <= atol + rtol * |oracle|


def torch_storage(arr, dtype, device):
    """numpy storage array (uint16 bf16 bits / float16 / float32) -> torch tensor on device."""
    import torch
    if dtype == inputs.BF16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)


def stack_layers(w, layers, with_cache=True):
    """Draw the given layers; returns list of LayerInputs and stacked numpy storage arrays."""
    lis = [inputs.layer_inputs(w, l, with_cache) for l in layers]
    q = np.stack([li.q for li in lis])
    k = np.stack([li.k for li in lis])
    kc = np.stack([li.k_cache for li in lis]) if with_cache else None
    vc = np.stack([li.v_cache for li in lis]) if with_cache else None
    return lis, q, k, kc, vc


def oracle_scores_layer(w, li):
    """float64 column sums [Hq, T] and lse [Hq, T] of one layer (all sequences)."""
    Hq, T = w.n_q_heads, w.total_tokens
    c = np.zeros((Hq, T))
    lse = np.zeros((Hq, T))
    cu = w.cu_seqlens
    for s in range(w.n_seqs):
        a, b = int(cu[s]), int(cu[s + 1])
        if b > a:
            cs, ls = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), w.causal)
            c[:, a:b], lse[:, a:b] = cs, ls
    return c, lse


def oracle_select_layer(w, scores32, b_imp, b_rep, sig_keep=None, anchor_mode=O.ANCHOR_ALTERNATE, explicit=None):
    """Signature + selection of one layer from float32 scores [Hq, T]; per-sequence results."""
    cu = w.cu_seqlens
    out = []
    for s in range(w.n_seqs):
        a, b = int(cu[s]), int(cu[s + 1])
        s32 = np.ascontiguousarray(scores32[:, a:b])
        keep = int(b_imp[s] + b_rep[s]) if sig_keep is None else int(sig_keep[s])
        theta = O.thresholds(s32, keep)
        sig = O.signatures(s32, theta)
        idx, kind = O.select(s32, sig, int(b_imp[s]), int(b_rep[s]), w.n_kv_heads, anchor_mode, explicit)
        out.append(dict(theta=theta, sig=sig, idx=idx, kind=kind))
    return out


def within_score_tolerance(g, o):
    return np.abs(g - o) <= SCORE_ATOL + SCORE_RTOL * np.abs(o)
