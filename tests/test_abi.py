"""The C-ABI library: it loads, exports every symbol the header declares, and rejects bad
arguments on the host before anything is launched (none of these calls touches a GPU)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2503_00022_b200 import binding as B
from paper_2503_00022_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    kbuild.build()
    return B.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "kvcrush.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvcrush_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared()
    assert set(B.EXPORTS) <= set(names) and len(names) >= 7
    for n in names:
        assert hasattr(lib, n), n
    assert B.kvcrush_version() >= 100
    assert B.strerror(B.ERR_WORKSPACE) == "workspace missing or too small"
    assert B.strerror(0) == "ok"


def _problem(**over):
    cu = np.asarray(over.pop("cu", [0, 100]), dtype=np.int32)
    kw = dict(n_layers=1, n_seqs=len(cu) - 1, n_q_heads=8, n_kv_heads=4, head_dim=64, total_tokens=int(cu[-1]),
              max_seqlen=int(np.diff(cu).max()), causal=1, softmax_scale=0.0, query_window=0,
              cu_seqlens_host=cu.ctypes.data, cu_seqlens_dev=0x1000)
    kw.update(over)
    p = B.ProblemStruct(**kw)
    p._keep = cu
    return p


def test_workspace_sizes_and_shape_validation(lib):
    out = ctypes.c_size_t(0)
    p = _problem()
    assert lib.kvcrush_workspace_size(ctypes.byref(p), B.STAGE_SCORE, ctypes.byref(out)) == 0
    assert out.value >= 8 * 100 * 4 and out.value % 256 == 0
    assert lib.kvcrush_workspace_size(ctypes.byref(p), B.STAGE_SELECT, ctypes.byref(out)) == 0
    assert out.value >= 100 * 12
    assert lib.kvcrush_workspace_size(ctypes.byref(p), B.STAGE_COMPACT, ctypes.byref(out)) == 0 and out.value == 0
    assert lib.kvcrush_workspace_size(ctypes.byref(p), 9, ctypes.byref(out)) == B.ERR_INVALID_ARG
    assert lib.kvcrush_workspace_size(None, 0, ctypes.byref(out)) == B.ERR_INVALID_ARG
    for bad in (dict(n_kv_heads=3), dict(n_layers=0), dict(total_tokens=99), dict(max_seqlen=50),
                dict(cu_seqlens_dev=None), dict(cu=[0, 60, 40]), dict(query_window=-1)):
        q = _problem(**bad)
        assert lib.kvcrush_workspace_size(ctypes.byref(q), 0, ctypes.byref(out)) == B.ERR_INVALID_ARG, bad
    assert lib.kvcrush_workspace_size(ctypes.byref(_problem(n_q_heads=256, n_kv_heads=256)), 0,
                                      ctypes.byref(out)) == B.ERR_UNSUPPORTED


def test_entry_points_reject_bad_arguments_before_launch(lib):
    p = _problem()
    t = B.TensorStruct(0x10000, B.BF16, 0, 100 * 8 * 64, 8 * 64, 64)
    odd = B.TensorStruct(0x10002, B.BF16, 0, 100 * 8 * 64, 8 * 64, 64)
    f16 = B.TensorStruct(0x10000, B.FP16, 0, 100 * 8 * 64, 8 * 64, 64)
    r = ctypes.byref
    # score: NULL outputs, misaligned tensor, dtype mismatch / unsupported, missing workspace
    assert lib.kvcrush_score(r(p), r(t), r(t), None, None, None, 0, 0, None, 0, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_score(r(p), r(odd), r(t), None, 0x100, None, 0, 0, 0x100, 1 << 20, 0x100, None) == B.ERR_MISALIGNED
    f32 = B.TensorStruct(0x10000, B.FP32, 0, 100 * 8 * 64, 8 * 64, 64)
    assert lib.kvcrush_score(r(p), r(f32), r(f32), None, 0x100, None, 0, B.SCORE_TENSOR, 0x100, 1 << 20, 0x100,
                             None) == B.ERR_UNSUPPORTED          # the tensor-core kernels take bf16 / fp16 only
    assert lib.kvcrush_score(r(p), r(t), r(f16), None, 0x100, None, 0, 0, 0x100, 1 << 20, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_score(r(p), r(t), r(t), None, 0x100, None, 0, 0, None, 0, 0x100, None) == B.ERR_WORKSPACE
    assert lib.kvcrush_score(r(p), r(t), r(t), None, 0x100, None, 0, 7, 0x100, 1 << 20, 0x100, None) == B.ERR_INVALID_ARG
    # signature: needs a rank or explicit thresholds; needs workspace when theta_out is NULL
    assert lib.kvcrush_signature(r(p), 0x100, None, None, 0x100, None, None, None, 0, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_signature(r(p), 0x100, 0x100, None, 0x100, None, None, None, 0, 0x100, None) == B.ERR_WORKSPACE
    # select: anchor mode range, explicit anchor needs bits, workspace
    assert lib.kvcrush_select(r(p), 0x100, None, 0x100, 0x100, 0x100, 5, None, 0, 0, 0, 0x100, 0x100, None, None, 0x100, 1 << 20,
                              0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_select(r(p), 0x100, None, 0x100, 0x100, 0x100, B.ANCHOR_EXPLICIT, None, 0, 0, 0, 0x100, 0x100, None,
                              None, 0x100, 1 << 20, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_select(r(p), 0x100, None, 0x100, 0x100, 0x100, 0, None, 0, 0, 0, 0x100, 0x100, None, None, 0x100, 16,
                              0x100, None) == B.ERR_WORKSPACE
    assert lib.kvcrush_select(r(p), 0x100, None, 0x100, 0x100, 0x100, 0, None, 0, 0, -1, 0x100, 0x100, None, None, 0x100, 1 << 20,
                              0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_select(r(p), 0x100, None, 0x100, 0x100, 0x100, 0, None, 0, -1, 0, 0x100, 0x100, None, None, 0x100, 1 << 20,
                              0x100, None) == B.ERR_INVALID_ARG
    # neither scores nor a ready importance array; a misaligned importance array
    assert lib.kvcrush_select(r(p), None, None, 0x100, 0x100, 0x100, 0, None, 0, 0, 0, 0x100, 0x100, None, None, 0x100,
                              1 << 20, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_select(r(p), None, 0x104, 0x100, 0x100, 0x100, 0, None, 0, 0, 0, 0x100, 0x100, None, None, 0x100,
                              1 << 20, 0x100, None) == B.ERR_MISALIGNED
    # page-granular select: page size, page vector too long, too many pages per sequence, workspace
    sp = lambda ps, prob=p, ws=1 << 20, ki=0: lib.kvcrush_select_pages(r(prob), 0x100, None, 0x100, ps, 0x100, 0x100, 0, None, 0,
                                                                       ki, 0, 0x100, 0x100, None, None, 0x100, ws, 0x100, None)
    assert sp(0) == B.ERR_INVALID_ARG
    assert sp(8, ki=-1) == B.ERR_INVALID_ARG
    assert sp(256) == B.ERR_UNSUPPORTED
    assert sp(8, ws=16) == B.ERR_WORKSPACE
    long_seq = _problem(cu=[0, 100000])
    assert sp(8, prob=long_seq, ws=1 << 30) == B.ERR_UNSUPPORTED
    assert lib.kvcrush_compact_pages(r(p), r(t), None, 0, 0x100, 0x100, 10, r(t), None, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_compact_pages(r(p), r(t), r(t), 8, 0x100, 0x100, 10, r(t), None, 0x100, None) == B.ERR_INVALID_ARG
    # decode step: NULL scores, dtype mismatch, misaligned tensor
    assert lib.kvcrush_score_decode(r(p), r(t), r(t), None, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_score_decode(r(p), r(t), r(f16), 0x100, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_score_decode(r(p), r(odd), r(t), 0x100, 0x100, None) == B.ERR_MISALIGNED
    # score gather: aliasing, negative counts
    assert lib.kvcrush_compact_scores(r(p), 0x100, 0, 0x100, 0x100, 4, 0x100, 16, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_compact_scores(r(p), 0x100, -1, 0x100, 0x100, 4, 0x200, 16, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_compact_scores(r(p), 0x100, 0, 0x100, 0x100, -4, 0x200, 16, 0x100, None) == B.ERR_INVALID_ARG
    # pooling: even kernel, aliasing
    assert lib.kvcrush_pool_scores(r(p), 0x100, 4, 0x200, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_pool_scores(r(p), 0x100, 3, 0x100, 0x100, None) == B.ERR_INVALID_ARG
    # compact: V without V_out, dtype mismatch, negative count
    assert lib.kvcrush_compact(r(p), r(t), r(t), 0x100, 0x100, 10, r(t), None, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_compact(r(p), r(t), None, 0x100, 0x100, 10, r(f16), None, 0x100, None) == B.ERR_INVALID_ARG
    assert lib.kvcrush_compact(r(p), r(t), None, 0x100, 0x100, -1, r(t), None, 0x100, None) == B.ERR_INVALID_ARG


def _no_cuda_device():
    import torch
    return not torch.cuda.is_available()


@pytest.mark.skipif(not _no_cuda_device(), reason="uses made-up device pointers: only where nothing can be launched")
def test_auto_does_not_drop_to_the_cuda_cores_when_the_driver_lacks_the_encoder(lib):
    """A problem the tensor-core kernels are made for (bf16, head_dim 64) on a machine whose driver cannot encode
    tensor maps (here: no driver at all): KVCRUSH_SCORE_AUTO and KVCRUSH_SCORE_TENSOR refuse with
    KVCRUSH_ERR_UNSUPPORTED instead of running the far slower CUDA-core kernels unnoticed.  A problem that the
    tensor-core kernels cannot take anyway (fp32, or a stride of 0 along the head axis) is not refused by AUTO for
    that reason: it goes on to the CUDA-core launch, which fails here for lack of a device."""
    p = _problem()
    r = ctypes.byref
    t = B.TensorStruct(0x10000, B.BF16, 0, 100 * 8 * 64, 8 * 64, 64)
    call = lambda q, k, impl, lse=None, ws=1 << 20: lib.kvcrush_score(r(p), r(q), r(k), lse, 0x100, None, 0, impl, 0x100,
                                                                      ws, 0x100, None)
    assert call(t, t, B.SCORE_AUTO) == B.ERR_UNSUPPORTED
    assert call(t, t, B.SCORE_TENSOR) == B.ERR_UNSUPPORTED
    f32 = B.TensorStruct(0x10000, B.FP32, 0, 100 * 8 * 64, 8 * 64, 64)
    assert call(f32, f32, B.SCORE_AUTO) == B.ERR_CUDA
    assert call(t, t, B.SCORE_SIMT) == B.ERR_CUDA
    # with the row log-sum-exp supplied the workspace only holds the work counters: 256 bytes are enough,
    # fewer are not; without it the full size is required
    assert call(t, t, B.SCORE_SIMT, lse=0x100, ws=256) == B.ERR_CUDA
    assert call(t, t, B.SCORE_SIMT, lse=0x100, ws=128) == B.ERR_WORKSPACE
    assert call(t, t, B.SCORE_SIMT, ws=256) == B.ERR_WORKSPACE


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()
