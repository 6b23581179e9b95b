"""TEST INFRASTRUCTURE - float64 CPU oracle for the KVCrush compression pass.

Not part of the product.  Only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import this module; it shares no code with the CUDA
library and never calls it.

Every function restates one step of the paper in plain numpy (the score step
can also run through the plain C routine in ``score_oracle.c`` which is the
same definition, row by row, for sizes numpy would be too slow for).  KVCrush is
a heuristic, so the oracle is the algorithm taken step by step:

  O1  A_h = softmax(Q_h K_h^T / sqrt(d_k))                     Algorithm 1
  O2  c_h(t) = sum_j A_h(j, t)   (w_h(t) = c_h(t) / S)          Algorithm 1, Sec. 3.1
  O3  theta_h, b_t[h] = [w_h(t) >= theta_h], packed             Algorithm 1, Sec. 3.1
  O4  B_important tokens by cumulative attention (H2O)         Sec. 3, Sec. 4.1.1
  O5  anchor a, d_t = Hamming(b_t, a)                           Algorithm 2, Sec. 3.2
  O6  B_representative buckets by d_t                           Algorithm 2, Sec. 3.2
  O7  representative = member closest to the bucket centroid   Algorithm 2, Sec. 3.2
  O8  kept = important U representatives                        Sec. 3.2
  O9  reduced cache = kept rows of K and V                      Sec. 3.2

Readings taken where the paper is silent or garbled (each one is a single
function or parameter here):

* column sums, not the row sums the printed index order would give (``scores``);
* theta_h is the k-th largest score of head h, k = total budget by default
  (``thresholds``) - PARITY UNPINNED by the paper: it only says the threshold
  keeps a target fraction of tokens per head;
* the importance of a token is the sum of its per-head scores, accumulated in
  float64 head by head in ascending order, KV group by KV group
  (``importance``); ties go to the lower token index;
* the tokens that are grouped are those NOT kept as important
  (``select``) - PARITY UNPINNED: Algorithm 2 lists all S tokens as input while
  Sec. 3 calls the representatives proxies of the evicted tokens;
* anchors: alternate = bit h is h mod 2; mean = per-bit majority over the
  grouped tokens, ties to 1; explicit bits cover "random" (``anchor_bits``)
  - the first bit of the alternating pattern and the population of the mean are
  PARITY UNPINNED;
* buckets are equal-frequency: sort the grouped tokens by (d_t, t) and cut the
  order into B_representative contiguous runs (``bucket_bounds``) - PARITY
  UNPINNED: the paper says "based on d_t" only, but d_t takes at most H+1
  values so only this reading yields exactly one representative per bucket and
  exactly B kept tokens;
* the centroid is the per-bit mean and "closest" is L1 (equivalently squared
  L2) distance, evaluated as an exact integer cost (``representative``).

SnapKV-style importance (Sec. 2.3 and Sec. 4.1.1 describe it in one sentence each: the
observation window is limited to the final tokens of the prompt, and max pooling keeps
neighbouring KVs) is covered by three small pieces, all PARITY UNPINNED by this paper
because it gives no formula for them:

* ``scores(..., rows=(L - w, L))``: only the last w queries vote;
* ``max_pool``: every per-head score becomes the maximum over a centred window of odd
  width (positions outside the sequence do not count);
* ``select(..., keep_recent=n)``: the last n tokens are important by decree (their
  importance is +inf) and count against B_important; ``keep_initial=n`` does the same for
  the first n tokens (Table 1 splits its 672-token budget into 32 initial + 512 middle +
  128 recent tokens).

Decode step (``decode_update``): the cumulative attention of H2O goes on while tokens are generated; one new query
adds its softmax row over the cached keys.  PARITY UNPINNED by this paper (it describes the baseline in a sentence).

Clustering baseline (``kmeans_select``; ablation "KMeans vs KVCrush", Fig. 3: k-means with 100 iterations in the place
of the anchor / bucket grouping): Lloyd's algorithm on the binary head vectors of the tokens that are not important,
k = B_representative, in exact rational arithmetic.  PARITY UNPINNED by the paper, which names the method and the
iteration count only: the initial centroids (the vectors at evenly spaced ranks of the grouped tokens), ties to the
lower cluster, empty clusters keeping their centroid, and the unused part of the budget going to the next most
important tokens are this file's readings.

Chunk- and page-granular eviction (Sec. 4.3.4: chunks of 8 tokens; Sec. 4.3.5: pages of 32 tokens): the
paper gives two sentences - the baseline sums the attention weights over a page, and the
binary vector of a page is the concatenation of the head vectors of its tokens.  Everything
else follows the token-level steps with a page in the place of a token
(``page_importance``, ``page_vectors``, ``select_pages``, ``compact_pages``).  PARITY UNPINNED:
a short last page counts its missing tokens as all-zero vectors of zero importance, and the
anchor of a page repeats the token anchor once per slot.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_C_SRC = os.path.join(_HERE, "score_oracle.c")
_C_LIB = os.path.join(_HERE, "libscore_oracle.so")

ANCHOR_ALTERNATE = 0
ANCHOR_MEAN = 1
ANCHOR_EXPLICIT = 2


# ---------------------------------------------------------------------------
# O1-O2  scores
# ---------------------------------------------------------------------------

def build_c(force: bool = False) -> str:
    """Compile ``score_oracle.c`` (gcc, OpenMP, no fast-math) next to its source."""
    if force or not os.path.exists(_C_LIB) or os.path.getmtime(_C_LIB) < os.path.getmtime(_C_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _C_LIB, _C_SRC, "-lm"])
    return _C_LIB


_lib = None


def _c_lib():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_c())
        lib.kvcrush_oracle_scores.restype = ctypes.c_int
        lib.kvcrush_oracle_scores.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        lib.kvcrush_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def n_threads() -> int:
    return int(_c_lib().kvcrush_oracle_threads())


def scores(q: np.ndarray, k: np.ndarray, causal: bool = True, scale: Optional[float] = None,
           normalize: bool = False, rows: Optional[Tuple[int, int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Column sums of the softmax attention matrix, one sequence (Algorithm 1).

    q [L, Hq, D], k [L, Hkv, D] float64.  Returns (c [Hq, L], lse [Hq, L]) float64;
    with ``normalize`` the first is w = c / L.  Runs the C routine (row by row).
    ``rows=(j0, j1)`` visits only the queries j0 <= j < j1: c is then the sum over those rows
    (the complete column sum for keys t >= j0 when causal) and lse is valid on those rows only.
    """
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    L, Hq, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == (L, Hkv, D) and Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    c = np.zeros((Hq, L), dtype=np.float64)
    lse = np.zeros((Hq, L), dtype=np.float64)
    j0, j1 = (0, L) if rows is None else (int(rows[0]), int(rows[1]))
    rc = _c_lib().kvcrush_oracle_scores(q.ctypes.data, k.ctypes.data, L, Hq, Hkv, D, int(bool(causal)),
                                        float(scale), j0, j1, c.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise RuntimeError("kvcrush_oracle_scores failed")
    if normalize and L > 0:
        c = c / L
    return c, lse


def attention_matrix(q: np.ndarray, k: np.ndarray, causal: bool = True,
                     scale: Optional[float] = None) -> np.ndarray:
    """Brute force: the explicit [Hq, L, L] softmax matrices A_h(j, t) (small L only)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    L, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    A = np.zeros((Hq, L, L), dtype=np.float64)
    for h in range(Hq):
        S = scale * (q[:, h, :] @ k[:, h // G, :].T)
        if causal:
            S = np.where(np.tril(np.ones((L, L), dtype=bool)), S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        E = np.exp(S)
        A[h] = E / E.sum(axis=1, keepdims=True)
    return A


def scores_bruteforce(q, k, causal=True, scale=None, normalize=False) -> np.ndarray:
    """c_h(t) = sum_j A_h(j, t) from the explicit matrices (small L only)."""
    A = attention_matrix(q, k, causal, scale)
    c = A.sum(axis=1)
    return c / q.shape[0] if normalize else c


def to_scores32(c: np.ndarray) -> np.ndarray:
    """The float32 array on which the signature and selection steps are defined."""
    return np.asarray(c, dtype=np.float64).astype(np.float32)


# ---------------------------------------------------------------------------
# O3  thresholds and signatures
# ---------------------------------------------------------------------------

def thresholds(scores32: np.ndarray, keep: int) -> np.ndarray:
    """theta_h = the ``keep``-th largest value of head h (Sec. 3.1: the threshold keeps
    a target fraction of the tokens of each head).  keep >= L -> -inf (all ones);
    keep <= 0 -> +inf (all zeros)."""
    Hq, L = scores32.shape
    if keep <= 0:
        return np.full(Hq, np.inf, dtype=np.float32)
    if keep >= L:
        return np.full(Hq, -np.inf, dtype=np.float32)
    srt = np.sort(scores32, axis=1)[:, ::-1]
    return np.ascontiguousarray(srt[:, keep - 1]).astype(np.float32)


def signatures(scores32: np.ndarray, theta: np.ndarray) -> np.ndarray:
    """b_t[h] = 1 iff score_h(t) >= theta_h (Algorithm 1), packed: head h is bit
    h mod 32 of word h div 32.  Returns uint32 [L, W]."""
    Hq, L = scores32.shape
    W = (Hq + 31) // 32
    sig = np.zeros((L, W), dtype=np.uint32)
    for h in range(Hq):
        bit = (scores32[h] >= np.float32(theta[h])).astype(np.uint32)
        sig[:, h // 32] |= bit << np.uint32(h % 32)
    return sig


# ---------------------------------------------------------------------------
# O4  importance (H2O)
# ---------------------------------------------------------------------------

def importance(scores32: np.ndarray, n_kv_heads: int) -> np.ndarray:
    """I(t): sum of the per-head scores, float64, heads added one at a time in
    ascending order inside each KV group, then the group sums in ascending order."""
    Hq, L = scores32.shape
    G = Hq // n_kv_heads
    total = np.zeros(L, dtype=np.float64)
    for g in range(n_kv_heads):
        group = np.zeros(L, dtype=np.float64)
        for h in range(g * G, (g + 1) * G):
            group = group + scores32[h].astype(np.float64)
        total = total + group
    return total


def max_pool(scores32: np.ndarray, kernel: int) -> np.ndarray:
    """out[h, t] = max of scores32[h, t - r .. t + r] inside the sequence, r = (kernel - 1) / 2,
    kernel odd (Sec. 2.3: max pooling retains the neighbours of a high-scoring token)."""
    assert kernel >= 1 and kernel % 2 == 1
    Hq, L = scores32.shape
    r = (kernel - 1) // 2
    out = np.empty_like(scores32)
    for t in range(L):
        out[:, t] = scores32[:, max(0, t - r):min(L, t + r + 1)].max(axis=1)
    return out


def top_important(I: np.ndarray, b_imp: int) -> np.ndarray:
    """Token ids of the b_imp largest I, ties to the lower index; returned ascending."""
    L = I.shape[0]
    order = np.lexsort((np.arange(L), -I))       # primary -I ascending, secondary index ascending
    return np.sort(order[: max(0, min(b_imp, L))]).astype(np.int64)


# ---------------------------------------------------------------------------
# O5  anchor and Hamming distance
# ---------------------------------------------------------------------------

def _head_mask(n_q_heads: int) -> np.ndarray:
    W = (n_q_heads + 31) // 32
    m = np.full(W, 0xFFFFFFFF, dtype=np.uint32)
    tail = n_q_heads - 32 * (W - 1)
    if tail < 32:
        m[-1] = np.uint32((1 << tail) - 1)
    return m


def unpack_bits(sig: np.ndarray, n_q_heads: int) -> np.ndarray:
    """[N, W] uint32 -> [N, Hq] array of 0/1."""
    N = sig.shape[0]
    out = np.zeros((N, n_q_heads), dtype=np.int64)
    for h in range(n_q_heads):
        out[:, h] = (sig[:, h // 32] >> np.uint32(h % 32)) & np.uint32(1)
    return out


def pack_bits(bits: np.ndarray) -> np.ndarray:
    n_q_heads = bits.shape[-1]
    W = (n_q_heads + 31) // 32
    out = np.zeros(W, dtype=np.uint32)
    for h in range(n_q_heads):
        if bits[h]:
            out[h // 32] |= np.uint32(1) << np.uint32(h % 32)
    return out


def anchor_bits(mode: int, n_q_heads: int, cand_sigs: Optional[np.ndarray] = None,
                explicit: Optional[np.ndarray] = None) -> np.ndarray:
    """Anchor a in {0,1}^H (Algorithm 2): alternating 0-1 (head 0 -> 0), per-bit mean of
    the grouped vectors rounded to a bit (ties -> 1), or caller-supplied bits."""
    if mode == ANCHOR_ALTERNATE:
        return pack_bits(np.arange(n_q_heads) % 2)
    if mode == ANCHOR_MEAN:
        bits = unpack_bits(cand_sigs, n_q_heads)
        N = bits.shape[0]
        return pack_bits((2 * bits.sum(axis=0) >= N).astype(np.int64))
    if mode == ANCHOR_EXPLICIT:
        return (np.asarray(explicit, dtype=np.uint32) & _head_mask(n_q_heads)).astype(np.uint32)
    raise ValueError(mode)


def hamming(sig: np.ndarray, anchor: np.ndarray, n_q_heads: int) -> np.ndarray:
    """d_t = number of heads on which b_t and a differ."""
    diff = unpack_bits(sig, n_q_heads) != unpack_bits(anchor[None, :], n_q_heads)
    return diff.sum(axis=1).astype(np.int64)


# ---------------------------------------------------------------------------
# O6-O7  buckets and representatives
# ---------------------------------------------------------------------------

def bucket_bounds(N: int, R: int) -> np.ndarray:
    """Equal-frequency cut of N sorted positions into R runs: run i is
    [floor(i*N/R), floor((i+1)*N/R))."""
    return np.asarray([(i * N) // R for i in range(R + 1)], dtype=np.int64)


def representative(member_tokens: np.ndarray, member_sigs: np.ndarray, n_q_heads: int) -> int:
    """The member whose vector is closest to the bucket centroid (Algorithm 2).

    Centroid c[h] = n_h / m.  For a 0/1 vector b, |b - c|_1 = sum_h c[h] + sum_{h: b[h]=1} (1 - 2 c[h]),
    so ranking by distance is ranking by the integer  sum_{h: b[h]=1} (m - 2 n_h).
    Ties go to the lower token index."""
    bits = unpack_bits(member_sigs, n_q_heads)
    m = bits.shape[0]
    n_h = bits.sum(axis=0)
    cost = (bits * (m - 2 * n_h)[None, :]).sum(axis=1)
    best = np.lexsort((member_tokens, cost))[0]
    return int(member_tokens[best])


# ---------------------------------------------------------------------------
# O4-O8  selection of the kept set of one sequence
# ---------------------------------------------------------------------------

def select(scores32: np.ndarray, sig: np.ndarray, b_imp: int, b_rep: int, n_kv_heads: int,
           anchor_mode: int = ANCHOR_ALTERNATE, explicit_anchor: Optional[np.ndarray] = None,
           keep_recent: int = 0, keep_initial: int = 0):
    """Kept token ids (ascending) and their kind (0 important, 1 representative).

    A budget b_imp + b_rep >= L keeps every token (kind 0).  The first keep_initial and the last
    keep_recent tokens are important by decree (Table 1: initial and recent parts of the budget)."""
    Hq, L = scores32.shape
    if b_imp + b_rep >= L:
        return np.arange(L, dtype=np.int64), np.zeros(L, dtype=np.uint8)
    I = importance(scores32, n_kv_heads)
    if keep_recent > 0 or keep_initial > 0:  # the observation window (SnapKV) / the attention sinks are kept
        I = I.copy()
        I[max(0, L - keep_recent):] = np.inf
        I[:min(L, keep_initial)] = np.inf
    imp = top_important(I, b_imp)
    is_imp = np.zeros(L, dtype=bool)
    is_imp[imp] = True
    reps = np.zeros(0, dtype=np.int64)
    if b_rep > 0:
        cand = np.nonzero(~is_imp)[0]
        N = cand.shape[0]
        a = anchor_bits(anchor_mode, Hq, sig[cand], explicit_anchor)
        d = hamming(sig[cand], a, Hq)
        order = np.lexsort((cand, d))                 # by d_t, then token index
        srt = cand[order]
        bounds = bucket_bounds(N, b_rep)
        reps = np.asarray([representative(srt[bounds[i]:bounds[i + 1]], sig[srt[bounds[i]:bounds[i + 1]]], Hq)
                           for i in range(b_rep)], dtype=np.int64)
    kept = np.sort(np.concatenate([imp, reps]))
    kind = np.zeros(kept.shape[0], dtype=np.uint8)
    kind[np.isin(kept, reps)] = 1
    return kept, kind


# ---------------------------------------------------------------------------
# Clustering baseline: k-means in the place of Algorithm 2's grouping (ablation "KMeans vs KVCrush", Fig. 3)
# ---------------------------------------------------------------------------

def kmeans_assign(bits: np.ndarray, cnt: np.ndarray, m: np.ndarray) -> np.ndarray:
    """Nearest centroid of every 0/1 row of ``bits`` [N, H]; centroid c is cnt[c] / m[c] (per-bit mean of m[c]
    vectors).  Squared Euclidean distance  sum_h (b_h - n_h/m)^2 = (sum_h n_h^2 + m * sum_{h: b_h=1} (m - 2 n_h)) / m^2
    is compared as an exact fraction (integers, cross-multiplied); ties go to the lower cluster index."""
    N, k = bits.shape[0], cnt.shape[0]
    out = np.zeros(N, dtype=np.int64)
    S = [int((cnt[c].astype(object) ** 2).sum()) for c in range(k)]
    wgt = [[int(m[c]) - 2 * int(x) for x in cnt[c]] for c in range(k)]
    for t in range(N):
        hs = np.nonzero(bits[t])[0]
        best_num, best_den, best_c = None, None, -1
        for c in range(k):
            mc = int(m[c])
            num = S[c] + mc * sum(wgt[c][h] for h in hs)        # distance = num / mc^2
            den = mc * mc
            if best_c < 0 or num * best_den < best_num * den:
                best_num, best_den, best_c = num, den, c
        out[t] = best_c
    return out


def kmeans_select(scores32: np.ndarray, sig: np.ndarray, b_imp: int, b_rep: int, n_kv_heads: int,
                  iterations: int = 100, keep_recent: int = 0, keep_initial: int = 0):
    """Kept token ids (ascending) and their kind when k-means takes the place of Algorithm 2's grouping.

    The important set is that of ``select``.  The other tokens (ascending, N of them) are clustered into
    k = b_rep clusters by Lloyd's algorithm on their binary head vectors: the initial centroids are the vectors at
    ranks floor(i*N/k); an iteration assigns every vector to its nearest centroid (``kmeans_assign``) and replaces
    each centroid by the per-bit mean of its members (a cluster without members keeps its centroid).  After
    ``iterations`` iterations one more assignment fixes the members; every cluster that has members contributes
    the member closest to its centroid (``representative``'s integer cost against that centroid, ties to the
    lower token).  Budget that empty clusters leave unused goes to the grouped tokens of largest importance that
    are not representatives (kind 0, like the important set)."""
    Hq, L = scores32.shape
    if b_imp + b_rep >= L:
        return np.arange(L, dtype=np.int64), np.zeros(L, dtype=np.uint8)
    I = importance(scores32, n_kv_heads)
    if keep_recent > 0 or keep_initial > 0:
        I = I.copy()
        I[max(0, L - keep_recent):] = np.inf
        I[:min(L, keep_initial)] = np.inf
    imp = top_important(I, b_imp)
    is_imp = np.zeros(L, dtype=bool)
    is_imp[imp] = True
    reps = np.zeros(0, dtype=np.int64)
    fill = np.zeros(0, dtype=np.int64)
    if b_rep > 0:
        cand = np.nonzero(~is_imp)[0]
        N, k = cand.shape[0], b_rep
        bits = unpack_bits(sig[cand], Hq).astype(np.int64)
        cnt = bits[[(i * N) // k for i in range(k)]].copy()
        m = np.ones(k, dtype=np.int64)
        for _ in range(iterations):
            assign = kmeans_assign(bits, cnt, m)
            for c in range(k):
                members = assign == c
                if members.any():
                    cnt[c] = bits[members].sum(axis=0)
                    m[c] = int(members.sum())
        assign = kmeans_assign(bits, cnt, m)
        rep_list = []
        for c in range(k):
            members = np.nonzero(assign == c)[0]
            if members.shape[0] == 0:
                continue
            cost = (bits[members] * (m[c] - 2 * cnt[c])[None, :]).sum(axis=1)
            rep_list.append(int(cand[members[np.lexsort((cand[members], cost))[0]]]))
        reps = np.asarray(sorted(rep_list), dtype=np.int64)
        shortfall = k - reps.shape[0]
        if shortfall > 0:
            rest = np.setdiff1d(cand, reps)
            fill = rest[top_important(I[rest], shortfall)]
    kept = np.sort(np.concatenate([imp, reps, fill]))
    kind = np.zeros(kept.shape[0], dtype=np.uint8)
    kind[np.isin(kept, reps)] = 1
    return kept, kind


# ---------------------------------------------------------------------------
# Page / chunk granularity (Sec. 4.3.4, Sec. 4.3.5)
# ---------------------------------------------------------------------------

def page_importance(I: np.ndarray, page_size: int) -> np.ndarray:
    """Importance of page p = sum of I(t) over its tokens, float64, added one token at a
    time in ascending order (Sec. 4.3.5: the baseline aggregates the attention sums per page)."""
    L = I.shape[0]
    n_pages = (L + page_size - 1) // page_size
    J = np.zeros(n_pages, dtype=np.float64)
    for i in range(page_size):
        t = np.arange(n_pages) * page_size + i
        ok = t < L
        J[ok] = J[ok] + I[t[ok]]
    return J


def page_vectors(sig: np.ndarray, page_size: int) -> np.ndarray:
    """Binary vector of a page = its tokens' head vectors one after the other (Sec. 4.3.5):
    uint32 [n_pages, page_size * W]; slots past the end of the sequence are zero."""
    L, W = sig.shape
    n_pages = (L + page_size - 1) // page_size
    out = np.zeros((n_pages * page_size, W), dtype=np.uint32)
    out[:L] = sig
    return out.reshape(n_pages, page_size * W)


def select_pages(scores32: np.ndarray, sig: np.ndarray, page_size: int, b_imp: int, b_rep: int,
                 n_kv_heads: int, anchor_mode: int = ANCHOR_ALTERNATE,
                 explicit_anchor: Optional[np.ndarray] = None, keep_recent: int = 0, keep_initial: int = 0):
    """Kept page ids (ascending) and their kind; budgets count pages.  The steps are those of
    ``select`` with pages for tokens: page importance, top b_imp pages, then Algorithm 2 on the
    page vectors of the other pages.  keep_initial / keep_recent count pages too."""
    Hq, L = scores32.shape
    W = sig.shape[1]
    n_pages = (L + page_size - 1) // page_size
    if b_imp + b_rep >= n_pages:
        return np.arange(n_pages, dtype=np.int64), np.zeros(n_pages, dtype=np.uint8)
    J = page_importance(importance(scores32, n_kv_heads), page_size)
    J[max(0, n_pages - keep_recent):] = np.inf
    J[:min(n_pages, keep_initial)] = np.inf
    imp = top_important(J, b_imp)
    is_imp = np.zeros(n_pages, dtype=bool)
    is_imp[imp] = True
    reps = np.zeros(0, dtype=np.int64)
    if b_rep > 0:
        n_bits = 32 * page_size * W              # unused bits of every word are zero on both sides
        vec = page_vectors(sig & _head_mask(Hq)[None, :], page_size)
        cand = np.nonzero(~is_imp)[0]
        N = cand.shape[0]
        if anchor_mode == ANCHOR_MEAN:
            a = anchor_bits(ANCHOR_MEAN, n_bits, vec[cand])
        else:
            a = np.tile(anchor_bits(anchor_mode, Hq, None, explicit_anchor), page_size)
        d = hamming(vec[cand], a, n_bits)
        srt = cand[np.lexsort((cand, d))]
        bounds = bucket_bounds(N, b_rep)
        reps = np.asarray([representative(srt[bounds[i]:bounds[i + 1]], vec[srt[bounds[i]:bounds[i + 1]]], n_bits)
                           for i in range(b_rep)], dtype=np.int64)
    kept = np.sort(np.concatenate([imp, reps]))
    kind = np.zeros(kept.shape[0], dtype=np.uint8)
    kind[np.isin(kept, reps)] = 1
    return kept, kind


def compact_pages(cache: np.ndarray, page_idx: np.ndarray, page_size: int) -> np.ndarray:
    """Reduced paged cache [n_kept, page_size, ...]: the kept pages of a token-major cache
    [L, ...]; the slots of a short last page are zero."""
    L = cache.shape[0]
    out = np.zeros((len(page_idx), page_size) + cache.shape[1:], dtype=cache.dtype)
    for i, p in enumerate(np.asarray(page_idx, dtype=np.int64)):
        n = min(page_size, L - int(p) * page_size)
        out[i, :n] = cache[int(p) * page_size:int(p) * page_size + n]
    return out


# ---------------------------------------------------------------------------
# Decode step of the cumulative attention (Sec. 2.3 / 4.1.1: H2O keeps summing attention weights while decoding)
# ---------------------------------------------------------------------------

def decode_update(scores: np.ndarray, q_new: np.ndarray, k: np.ndarray, scale: Optional[float] = None) -> np.ndarray:
    """scores [Hq, L] (float64) plus the attention row of one new query q_new [Hq, D] over all L cached keys
    k [L, Hkv, D] (the new token's own key is the last one): A_h(t) = softmax_t(q_h . k_t / sqrt(d_k))."""
    Hq, D = q_new.shape
    L, Hkv, _ = k.shape
    G = Hq // Hkv
    sc = (1.0 / np.sqrt(D)) if scale is None else float(scale)
    out = np.array(scores, dtype=np.float64, copy=True)
    for h in range(Hq):
        logits = (k[:, h // G, :].astype(np.float64) @ q_new[h].astype(np.float64)) * sc
        e = np.exp(logits - logits.max())
        out[h] += e / e.sum()
    return out


def compact(cache: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Reduced cache: rows idx of a token-major cache [L, ...] (byte copy)."""
    return np.ascontiguousarray(cache[np.asarray(idx, dtype=np.int64)])


def compress_sequence(q, k, b_imp, b_rep, sig_keep=None, causal=True, scale=None,
                      anchor_mode=ANCHOR_ALTERNATE, explicit_anchor=None):
    """The whole pass for one sequence of one layer. q [L,Hq,D], k [L,Hkv,D] float64."""
    c, lse = scores(q, k, causal, scale)
    s32 = to_scores32(c)
    keep = (b_imp + b_rep) if sig_keep is None else sig_keep
    theta = thresholds(s32, keep)
    sig = signatures(s32, theta)
    idx, kind = select(s32, sig, b_imp, b_rep, k.shape[1], anchor_mode, explicit_anchor)
    return dict(colsum=c, lse=lse, scores32=s32, theta=theta, sig=sig, idx=idx, kind=kind)


# ---------------------------------------------------------------------------
# Eq. 1
# ---------------------------------------------------------------------------

def kv_memory_bytes(batch: int, n_layers: int, n_heads: int, seq_len: int, head_dim: int,
                    precision_bytes: int) -> int:
    """Eq. 1: 2 * B * N_L * N_H * L_seq * D * precision."""
    return 2 * batch * n_layers * n_heads * seq_len * head_dim * precision_bytes
