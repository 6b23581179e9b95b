"""ctypes binding of libkvcrush.so: the same names as the C ABI (include/kvcrush.h).

Only argument marshalling lives here.  torch is used to own device memory and to
name the CUDA stream; every step of the compression pass runs inside the library's
kernels.  There is no CPU fallback: if the library cannot be loaded the first call
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvcrush.so")

# constants of include/kvcrush.h
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_WORKSPACE, ERR_CUDA = 0, -1, -2, -3, -4, -5
ERR_STATIC_LIMIT = -6
STATIC_THETA_MAX = 65536
DEV_OK, DEV_TIMEOUT, DEV_BUDGET = 0, 1, 2
BF16, FP16, FP32 = 0, 1, 2
STAGE_SCORE, STAGE_SIGNATURE, STAGE_SELECT, STAGE_COMPACT = 0, 1, 2, 3
ANCHOR_ALTERNATE, ANCHOR_MEAN, ANCHOR_EXPLICIT = 0, 1, 2
SCORE_AUTO, SCORE_SIMT, SCORE_TENSOR = 0, 1, 2

EXPORTS = ("kvcrush_workspace_size", "kvcrush_score", "kvcrush_signature", "kvcrush_select",
           "kvcrush_compact", "kvcrush_strerror", "kvcrush_version", "kvcrush_signature_static",
           "kvcrush_pool_scores", "kvcrush_select_pages", "kvcrush_compact_pages", "kvcrush_score_decode",
           "kvcrush_compact_scores", "kvcrush_kmeans_workspace_size", "kvcrush_kmeans_select")


class ProblemStruct(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("n_seqs", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("total_tokens", ctypes.c_int32),
        ("max_seqlen", ctypes.c_int32), ("causal", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("query_window", ctypes.c_int32), ("cu_seqlens_host", ctypes.c_void_p), ("cu_seqlens_dev", ctypes.c_void_p),
    ]


class TensorStruct(ctypes.Structure):
    _fields_ = [
        ("ptr_dev", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("stride_layer", ctypes.c_int64), ("stride_token", ctypes.c_int64), ("stride_head", ctypes.c_int64),
    ]


class KvcrushError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if libkvcrush.so has not been built (python -m paper_2503_00022_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2503_00022_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
        P, T = ctypes.POINTER(ProblemStruct), ctypes.POINTER(TensorStruct)
        L.kvcrush_workspace_size.argtypes = [P, i32, ctypes.POINTER(sz)]
        L.kvcrush_score.argtypes = [P, T, T, vp, vp, vp, i32, i32, vp, sz, vp, vp]
        L.kvcrush_score_decode.argtypes = [P, T, T, vp, vp, vp]
        L.kvcrush_compact_scores.argtypes = [P, vp, i32, vp, vp, i64, vp, i64, vp, vp]
        L.kvcrush_signature.argtypes = [P, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.kvcrush_select.argtypes = [P, vp, vp, vp, vp, vp, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.kvcrush_pool_scores.argtypes = [P, vp, i32, vp, vp, vp]
        L.kvcrush_kmeans_workspace_size.argtypes = [P, i32, ctypes.POINTER(sz)]
        L.kvcrush_kmeans_select.argtypes = [P, vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.kvcrush_compact.argtypes = [P, T, T, vp, vp, i64, T, T, vp, vp]
        L.kvcrush_select_pages.argtypes = [P, vp, vp, vp, i32, vp, vp, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.kvcrush_compact_pages.argtypes = [P, T, T, i32, vp, vp, i64, T, T, vp, vp]
        L.kvcrush_signature_static.argtypes = [P, vp, vp, vp, vp, vp]
        L.kvcrush_strerror.argtypes = [i32]
        L.kvcrush_strerror.restype = ctypes.c_char_p
        L.kvcrush_version.argtypes = []
        for name in EXPORTS:
            if name != "kvcrush_strerror":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().kvcrush_strerror(int(code)).decode()


def kvcrush_version() -> int:
    return int(lib().kvcrush_version())


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise KvcrushError(rc, where)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream() -> int:
    import torch
    return int(torch.cuda.current_stream().cuda_stream)


def dtype_code(torch_dtype) -> int:
    import torch
    return {torch.bfloat16: BF16, torch.float16: FP16, torch.float32: FP32}[torch_dtype]


class Problem:
    """Owns a kvcrush_problem_t plus the host and device copies of cu_seqlens it points at."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 seqlens: Sequence[int], causal: bool = True, softmax_scale: float = 0.0, device="cuda:0",
                 query_window: int = 0):
        import torch
        self.seqlens = tuple(int(x) for x in seqlens)
        self.cu_host = np.zeros(len(self.seqlens) + 1, dtype=np.int32)
        self.cu_host[1:] = np.cumsum(np.asarray(self.seqlens, dtype=np.int64))
        self.cu_dev = torch.from_numpy(self.cu_host).to(device)
        self.device = self.cu_dev.device
        self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        self.n_seqs = len(self.seqlens)
        self.total_tokens = int(self.cu_host[-1])
        self.max_seqlen = max(self.seqlens) if self.seqlens else 0
        self.W = (n_q_heads + 31) // 32
        self.struct = ProblemStruct(
            n_layers, self.n_seqs, n_q_heads, n_kv_heads, head_dim, self.total_tokens, self.max_seqlen,
            int(causal), float(softmax_scale), int(query_window), self.cu_host.ctypes.data, int(self.cu_dev.data_ptr()))

    @property
    def ref(self):
        return ctypes.byref(self.struct)


def tensor_struct(t) -> TensorStruct:
    """Descriptor of a torch tensor viewed as [n_layers, tokens, heads, head_dim] (last stride 1)."""
    assert t.dim() == 4 and t.stride(3) == 1, "expected [layers, tokens, heads, D] with contiguous D"
    return TensorStruct(int(t.data_ptr()), dtype_code(t.dtype), 0, t.stride(0), t.stride(1), t.stride(2))


def kvcrush_workspace_size(problem: Problem, stage: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().kvcrush_workspace_size(problem.ref, stage, ctypes.byref(out)), "kvcrush_workspace_size")
    return int(out.value)


def kvcrush_score(problem: Problem, q, k, scores, *, lse_in=None, lse_out=None, normalize=False,
                  impl=SCORE_AUTO, workspace=None, status=None, stream: Optional[int] = None) -> None:
    qs, ks = tensor_struct(q), tensor_struct(k)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().kvcrush_score(problem.ref, ctypes.byref(qs), ctypes.byref(ks), _ptr(lse_in), _ptr(scores),
                               _ptr(lse_out), int(normalize), int(impl), _ptr(workspace), ws_bytes, _ptr(status),
                               _stream() if stream is None else stream), "kvcrush_score")


def kvcrush_score_decode(problem: Problem, q_new, k, scores, *, status=None, stream: Optional[int] = None) -> None:
    """Adds the attention row of every sequence's new query (q_new [layers, n_seqs, Hq, D]) to the running scores."""
    qs, ks = tensor_struct(q_new), tensor_struct(k)
    _check(lib().kvcrush_score_decode(problem.ref, ctypes.byref(qs), ctypes.byref(ks), _ptr(scores), _ptr(status),
                                      _stream() if stream is None else stream), "kvcrush_score_decode")


def kvcrush_compact_scores(problem: Problem, scores_in, page_size: int, cu_kept, idx, total_kept: int, scores_out, *,
                           status=None, stream: Optional[int] = None) -> None:
    """Gathers running scores [layers, Hq, T] along the kept tokens (page_size 0) or pages into scores_out
    [layers, Hq, T_out], arranged like the reduced cache."""
    _check(lib().kvcrush_compact_scores(problem.ref, _ptr(scores_in), int(page_size), _ptr(cu_kept), _ptr(idx),
                                        int(total_kept), _ptr(scores_out), int(scores_out.shape[-1]), _ptr(status),
                                        _stream() if stream is None else stream), "kvcrush_compact_scores")


def kvcrush_signature(problem: Problem, scores, sigs, *, sig_keep=None, theta_in=None, theta_out=None,
                      importance_out=None, workspace=None, status=None, stream: Optional[int] = None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().kvcrush_signature(problem.ref, _ptr(scores), _ptr(sig_keep), _ptr(theta_in), _ptr(sigs),
                                   _ptr(theta_out), _ptr(importance_out), _ptr(workspace), ws_bytes, _ptr(status),
                                   _stream() if stream is None else stream), "kvcrush_signature")


def kvcrush_signature_static(problem: Problem, scores, sigs, sig_keep, *, status=None,
                             stream: Optional[int] = None) -> None:
    """kvcrush_signature without a workspace: the thresholds' scratch is device memory built into the
    library (at most STATIC_THETA_MAX thresholds).  For hosts that must not allocate; calls on one
    device must not overlap."""
    _check(lib().kvcrush_signature_static(problem.ref, _ptr(scores), _ptr(sig_keep), _ptr(sigs), _ptr(status),
                                          _stream() if stream is None else stream), "kvcrush_signature_static")


def kvcrush_select(problem: Problem, scores, sigs, budget_imp, budget_rep, cu_kept, idx, *, importance=None,
                   kind=None, n_kept=None, anchor_mode=ANCHOR_ALTERNATE, anchor_bits=None, anchor_per_segment=False, keep_recent=0,
                   keep_initial=0, workspace=None, status=None, stream: Optional[int] = None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().kvcrush_select(problem.ref, _ptr(scores), _ptr(importance), _ptr(sigs), _ptr(budget_imp), _ptr(budget_rep),
                                int(anchor_mode), _ptr(anchor_bits), int(anchor_per_segment), int(keep_initial),
                                int(keep_recent), _ptr(cu_kept),
                                _ptr(idx), _ptr(kind), _ptr(n_kept), _ptr(workspace), ws_bytes, _ptr(status),
                                _stream() if stream is None else stream), "kvcrush_select")


def kvcrush_kmeans_workspace_size(problem: Problem, max_budget_rep: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().kvcrush_kmeans_workspace_size(problem.ref, int(max_budget_rep), ctypes.byref(out)),
           "kvcrush_kmeans_workspace_size")
    return int(out.value)


def kvcrush_kmeans_select(problem: Problem, scores, sigs, budget_imp, budget_rep, max_budget_rep: int, iterations: int,
                          cu_kept, idx, *, importance=None, kind=None, n_kept=None, keep_initial=0, keep_recent=0,
                          workspace=None, status=None, stream: Optional[int] = None) -> None:
    """The clustering baseline: k-means on the binary head vectors in the place of kvcrush_select's grouping."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().kvcrush_kmeans_select(problem.ref, _ptr(scores), _ptr(importance), _ptr(sigs), _ptr(budget_imp),
                                       _ptr(budget_rep), int(max_budget_rep), int(iterations), int(keep_initial),
                                       int(keep_recent), _ptr(cu_kept), _ptr(idx), _ptr(kind), _ptr(n_kept),
                                       _ptr(workspace), ws_bytes, _ptr(status),
                                       _stream() if stream is None else stream), "kvcrush_kmeans_select")


def kvcrush_pool_scores(problem: Problem, scores_in, kernel: int, scores_out, *, status=None,
                        stream: Optional[int] = None) -> None:
    _check(lib().kvcrush_pool_scores(problem.ref, _ptr(scores_in), int(kernel), _ptr(scores_out), _ptr(status),
                                     _stream() if stream is None else stream), "kvcrush_pool_scores")


def kvcrush_compact(problem: Problem, k, v, cu_kept, idx, total_kept: int, k_out, v_out, *, status=None,
                    stream: Optional[int] = None) -> None:
    ks, kos = tensor_struct(k), tensor_struct(k_out)
    vs = tensor_struct(v) if v is not None else None
    vos = tensor_struct(v_out) if v_out is not None else None
    _check(lib().kvcrush_compact(problem.ref, ctypes.byref(ks), ctypes.byref(vs) if vs is not None else None,
                                 _ptr(cu_kept), _ptr(idx), int(total_kept), ctypes.byref(kos),
                                 ctypes.byref(vos) if vos is not None else None, _ptr(status),
                                 _stream() if stream is None else stream), "kvcrush_compact")


def kvcrush_select_pages(problem: Problem, scores, sigs, page_size: int, budget_imp, budget_rep, cu_kept, page_idx, *,
                         importance=None, kind=None, n_kept=None, anchor_mode=ANCHOR_ALTERNATE, anchor_bits=None,
                         anchor_per_segment=False,
                         keep_initial=0, keep_recent=0, workspace=None, status=None,
                         stream: Optional[int] = None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().kvcrush_select_pages(problem.ref, _ptr(scores), _ptr(importance), _ptr(sigs), int(page_size), _ptr(budget_imp),
                                      _ptr(budget_rep), int(anchor_mode), _ptr(anchor_bits), int(anchor_per_segment),
                                      int(keep_initial), int(keep_recent), _ptr(cu_kept), _ptr(page_idx), _ptr(kind), _ptr(n_kept),
                                      _ptr(workspace), ws_bytes,
                                      _ptr(status), _stream() if stream is None else stream), "kvcrush_select_pages")


def kvcrush_compact_pages(problem: Problem, k, v, page_size: int, cu_kept, page_idx, total_kept_pages: int, k_out,
                          v_out, *, status=None, stream: Optional[int] = None) -> None:
    ks, kos = tensor_struct(k), tensor_struct(k_out)
    vs = tensor_struct(v) if v is not None else None
    vos = tensor_struct(v_out) if v_out is not None else None
    _check(lib().kvcrush_compact_pages(problem.ref, ctypes.byref(ks), ctypes.byref(vs) if vs is not None else None,
                                       int(page_size), _ptr(cu_kept), _ptr(page_idx), int(total_kept_pages),
                                       ctypes.byref(kos), ctypes.byref(vos) if vos is not None else None,
                                       _ptr(status), _stream() if stream is None else stream), "kvcrush_compact_pages")


class CompressionPass:
    """All buffers of one compression pass, allocated once; ``run`` enqueues the four stages.

    q [Lyr, T, Hq, D], k [Lyr, T, Hkv, D] (scoring inputs) and the K/V caches are the caller's
    tensors; budgets are per (layer, sequence) numpy arrays.  Nothing here computes: it
    sizes and allocates outputs and workspaces and forwards pointers.

    page_size > 0 selects and gathers whole pages of that many tokens: budgets then count pages,
    ``idx`` holds page numbers, the reduced cache has page_size rows per kept page and keep_initial /
    keep_recent count pages as well.
    """

    def __init__(self, problem: Problem, budget_imp: np.ndarray, budget_rep: np.ndarray,
                 cache_dtype=None, sig_keep: Optional[np.ndarray] = None, anchor_mode=ANCHOR_ALTERNATE,
                 anchor_bits: Optional[np.ndarray] = None, impl=SCORE_AUTO, with_kind=True, with_cache=True,
                 pool_kernel: int = 0, keep_recent: int = 0, page_size: int = 0, keep_initial: int = 0,
                 share_importance: bool = True):
        import torch
        self.page_size = int(page_size)
        unit = max(self.page_size, 1)
        p = self.problem = problem
        dev = p.device
        Lyr, S, T = p.n_layers, p.n_seqs, p.total_tokens
        bi = np.broadcast_to(np.asarray(budget_imp, dtype=np.int32), (Lyr, S)).copy()
        br = np.broadcast_to(np.asarray(budget_rep, dtype=np.int32), (Lyr, S)).copy()
        lens = (np.asarray(p.seqlens, dtype=np.int64)[None, :] + unit - 1) // unit       # tokens, or pages
        kept = np.minimum(bi.astype(np.int64) + br, lens)
        cu_kept = np.zeros(Lyr * S + 1, dtype=np.int64)
        cu_kept[1:] = np.cumsum(kept.reshape(-1))
        self.kept_per_layer = kept.sum(axis=1)
        self.total_kept = int(cu_kept[-1])
        self.cu_kept_host = cu_kept.astype(np.int32)
        keep = (bi + br) * unit if sig_keep is None else np.broadcast_to(np.asarray(sig_keep, dtype=np.int32), (Lyr, S))
        self.budget_imp = torch.from_numpy(bi).to(dev)
        self.budget_rep = torch.from_numpy(br).to(dev)
        self.sig_keep = torch.from_numpy(np.array(keep, dtype=np.int32, copy=True)).to(dev)
        self.cu_kept = torch.from_numpy(self.cu_kept_host).to(dev)
        self.anchor_mode = anchor_mode
        self.anchor_bits = None if anchor_bits is None else torch.from_numpy(
            np.ascontiguousarray(anchor_bits, dtype=np.uint32).view(np.int32)).to(dev)
        self.impl = impl
        self.pool_kernel, self.keep_recent, self.keep_initial = int(pool_kernel), int(keep_recent), int(keep_initial)
        self.pooled = None
        self.scores = torch.empty((Lyr, p.n_q_heads, T), dtype=torch.float32, device=dev)
        self.lse = torch.empty((Lyr, p.n_q_heads, T), dtype=torch.float32, device=dev)
        if self.pool_kernel > 1:
            self.pooled = torch.empty((Lyr, p.n_q_heads, T), dtype=torch.float32, device=dev)
        self.theta = torch.empty((Lyr, S, p.n_q_heads), dtype=torch.float32, device=dev)
        self.sigs = torch.empty((Lyr, T, p.W), dtype=torch.int32, device=dev)
        self.idx = torch.empty((max(self.total_kept, 1),), dtype=torch.int32, device=dev)
        self.kind = torch.empty((max(self.total_kept, 1),), dtype=torch.uint8, device=dev) if with_kind else None
        self.n_kept = torch.empty((Lyr, S), dtype=torch.int32, device=dev)
        # token importance handed from the signature stage to the selection stage (one pass over the scores saved)
        self.importance = torch.empty((Lyr, T), dtype=torch.float64, device=dev) if share_importance else None
        self._importance_of = None          # data pointer of the scores the importance was computed from
        self.status = torch.zeros(4, dtype=torch.int32, device=dev)
        nbytes = max(kvcrush_workspace_size(p, st) for st in (STAGE_SCORE, STAGE_SIGNATURE, STAGE_SELECT))
        self.workspace = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=dev)
        self.k_out = self.v_out = None
        if with_cache and cache_dtype is not None:
            n_out = int(self.kept_per_layer.max()) * unit if Lyr else 0
            shape = (Lyr, max(n_out, 1), p.n_kv_heads, p.head_dim)
            self.k_out = torch.empty(shape, dtype=cache_dtype, device=dev)
            self.v_out = torch.empty(shape, dtype=cache_dtype, device=dev)

    def score(self, q, k, lse_in=None):
        kvcrush_score(self.problem, q, k, self.scores, lse_in=lse_in, lse_out=None if lse_in is not None else self.lse,
                      impl=self.impl, workspace=self.workspace, status=self.status)

    def pool(self):
        """Max-pools self.scores into self.pooled, which signature/select then use."""
        kvcrush_pool_scores(self.problem, self.scores, self.pool_kernel, self.pooled, status=self.status)

    def _selection_scores(self, scores):
        if scores is not None:
            return scores
        return self.pooled if self.pooled is not None else self.scores

    def signature(self, scores=None):
        sc = self._selection_scores(scores)
        kvcrush_signature(self.problem, sc, self.sigs, sig_keep=self.sig_keep, theta_out=self.theta,
                          importance_out=self.importance, workspace=self.workspace, status=self.status)
        self._importance_of = None if self.importance is None else int(sc.data_ptr())

    def select(self, scores=None):
        sc = self._selection_scores(scores)
        imp = self.importance if self._importance_of == int(sc.data_ptr()) else None
        if self.page_size:
            kvcrush_select_pages(self.problem, sc, self.sigs, self.page_size, importance=imp,
                                 budget_imp=self.budget_imp, budget_rep=self.budget_rep, cu_kept=self.cu_kept,
                                 page_idx=self.idx, kind=self.kind,
                                 n_kept=self.n_kept, anchor_mode=self.anchor_mode, anchor_bits=self.anchor_bits,
                                 keep_initial=self.keep_initial, keep_recent=self.keep_recent,
                                 workspace=self.workspace, status=self.status)
            return
        kvcrush_select(self.problem, sc, self.sigs, self.budget_imp,
                       self.budget_rep, self.cu_kept, self.idx, importance=imp, kind=self.kind, n_kept=self.n_kept,
                       anchor_mode=self.anchor_mode,
                       anchor_bits=self.anchor_bits, keep_recent=self.keep_recent, keep_initial=self.keep_initial,
                       workspace=self.workspace, status=self.status)

    def compact(self, k_cache, v_cache):
        if self.page_size:
            kvcrush_compact_pages(self.problem, k_cache, v_cache, self.page_size, self.cu_kept, self.idx,
                                  self.total_kept, self.k_out, self.v_out, status=self.status)
            return
        kvcrush_compact(self.problem, k_cache, v_cache, self.cu_kept, self.idx, self.total_kept, self.k_out,
                        self.v_out, status=self.status)

    def run(self, q, k, k_cache=None, v_cache=None, lse_in=None):
        self.score(q, k, lse_in)
        if self.pooled is not None:
            self.pool()
        self.signature()
        self.select()
        if k_cache is not None:
            self.compact(k_cache, v_cache)

    def capture(self, q, k, k_cache=None, v_cache=None, lse_in=None):
        """Records one ``run`` into a CUDA graph: the library only enqueues kernels and one memset on the stream
        it is given, so the whole pass replays as a single launch (worth it when the pass is short and launch
        overhead shows).  The tensors must stay where they are; ``replay`` runs the pass on their current contents."""
        import torch
        self.run(q, k, k_cache, v_cache, lse_in)          # outside the capture: one-time kernel attribute calls
        torch.cuda.synchronize()
        self.check_status()
        self._graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self._graph):
            self.run(q, k, k_cache, v_cache, lse_in)
        return self._graph

    def replay(self):
        self._graph.replay()

    def check_status(self):
        st = self.status.cpu().tolist()
        if st[0] != DEV_OK:
            raise RuntimeError(f"kvcrush device error {st}")

    def kept(self, layer: int, seq: int) -> np.ndarray:
        """Kept token ids (page numbers when page_size > 0; host copy) of one (layer, sequence)."""
        seg = layer * self.problem.n_seqs + seq
        lo, hi = int(self.cu_kept_host[seg]), int(self.cu_kept_host[seg + 1])
        return self.idx[lo:hi].cpu().numpy()
