"""Seeded synthetic workloads for the KV-cache compression pass.

This module only draws random tensors and rounds them to their storage type.
It contains none of the method's arithmetic (no softmax, no scores, no
selection) so that the CPU oracle and the CUDA path can both be fed from it
without sharing any computation.

Recipe (one layer at a time, ``seed = base_seed + layer``, numpy Philox):

* Q, K, V ~ N(0, 1) drawn in float32, token-major ``[T, heads, D]``;
* inside every sequence the key rows of tokens 0..3 are multiplied by 4
  ("attention sinks") and a seeded random subset of the remaining tokens by 2
  ("heavy hitters"); the same token set is used for all heads of the layer;
* the arrays are rounded ONCE to the storage type (bf16 round-to-nearest-even
  for Q/K scoring inputs, fp16 for a separate K/V cache, or kept in fp32) and
  those rounded values are what both sides consume.

The workloads mirror long-prompt KV-cache compression at a fixed total budget
(the paper evaluates prompts of roughly 2k-18k tokens with a 2048-token cache
budget, Table 3 / Table 1); no benchmark-suite item is reproduced here.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

BF16 = "bf16"
FP16 = "fp16"
FP32 = "fp32"

SINK_TOKENS = 4
SINK_GAIN = 4.0
HEAVY_GAIN = 2.0


@dataclass(frozen=True)
class Workload:
    """Shape of one compression workload (all layers share the shape)."""

    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seqlens: Tuple[int, ...]            # one entry per sequence of the batch
    qk_dtype: str                       # storage type of the scoring Q / K
    cache_dtype: str                    # storage type of the K/V cache that is compacted
    budget_fraction: float              # total budget B = floor(fraction * L) unless budget is set
    budget: Optional[int] = None        # fixed total budget for every sequence
    heavy_fraction: Tuple[float, float] = (0.05, 0.05)   # (lo, hi): per-layer U[lo, hi]
    base_seed: int = 1000
    causal: bool = True

    @property
    def n_seqs(self) -> int:
        return len(self.seqlens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    @property
    def max_seqlen(self) -> int:
        return int(max(self.seqlens)) if self.seqlens else 0

    @property
    def cu_seqlens(self) -> np.ndarray:
        out = np.zeros(self.n_seqs + 1, dtype=np.int32)
        out[1:] = np.cumsum(np.asarray(self.seqlens, dtype=np.int64))
        return out

    def budgets(self) -> Tuple[np.ndarray, np.ndarray]:
        """Per-sequence (B_important, B_representative): B_rep = floor(B/2), B_imp = B - B_rep."""
        imp, rep = [], []
        for L in self.seqlens:
            B = self.budget if self.budget is not None else int(np.floor(self.budget_fraction * L))
            B = min(B, L)
            r = B // 2
            imp.append(B - r)
            rep.append(r)
        return np.asarray(imp, dtype=np.int32), np.asarray(rep, dtype=np.int32)


def _ragged_lengths(n: int, lo: int, hi: int, seed: int) -> Tuple[int, ...]:
    g = np.random.Generator(np.random.Philox(seed))
    return tuple(int(x) for x in g.integers(lo, hi + 1, size=n))


def paper_workloads() -> Dict[str, Workload]:
    """The five benchmark shapes (small -> large)."""
    return {
        "cfg1_small_fp32": Workload(
            "cfg1_small_fp32", 1, 8, 8, 64, (512,), FP32, FP32, 0.25, budget=128, base_seed=1100),
        "cfg2_llama2_layer_4k": Workload(
            "cfg2_llama2_layer_4k", 1, 32, 32, 128, (4096,), BF16, BF16, 0.25, budget=1024, base_seed=1200),
        "cfg3_llama2_32l_8k": Workload(
            "cfg3_llama2_32l_8k", 32, 32, 32, 128, (8192,), BF16, FP16, 0.25, budget=2048,
            heavy_fraction=(0.02, 0.10), base_seed=1300),
        "cfg4_llama3_gqa_32k": Workload(
            "cfg4_llama3_gqa_32k", 32, 32, 8, 128, (32768,), BF16, BF16, 0.20, budget=6554, base_seed=1400),
        "cfg5_ragged_batch16": Workload(
            "cfg5_ragged_batch16", 32, 32, 32, 128, _ragged_lengths(16, 1024, 4096, 1500), BF16, BF16,
            0.25, base_seed=1500),
    }


def shrink(w: Workload, n_layers: int) -> Workload:
    """Same shape with fewer layers (used by tests and by bounded CPU samples)."""
    return replace(w, n_layers=n_layers, name=f"{w.name}[{n_layers}L]")


# ---------------------------------------------------------------------------
# storage-type rounding (bit manipulation only)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array -> array in its storage representation.

    bf16 -> uint16 bit patterns, fp16 -> numpy float16, fp32 -> float32.
    """
    if dtype == BF16:
        try:                                     # same rounding, multi-threaded
            import torch
            t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
            return t.view(torch.int16).numpy().view(np.uint16)
        except ImportError:
            return f32_to_bf16_bits(x)
    if dtype == FP16:
        return x.astype(np.float16)
    if dtype == FP32:
        return np.ascontiguousarray(x, dtype=np.float32)
    raise ValueError(dtype)


def widen(x: np.ndarray, dtype: str) -> np.ndarray:
    """Storage representation -> float64 (exact)."""
    if dtype == BF16:
        return bf16_bits_to_f32(x).astype(np.float64)
    return x.astype(np.float64)


def storage_itemsize(dtype: str) -> int:
    return {BF16: 2, FP16: 2, FP32: 4}[dtype]


# ---------------------------------------------------------------------------
# per-layer generation
# ---------------------------------------------------------------------------

@dataclass
class LayerInputs:
    q: np.ndarray            # [T, Hq, D]  storage of qk_dtype
    k: np.ndarray            # [T, Hkv, D] storage of qk_dtype
    k_cache: np.ndarray      # [T, Hkv, D] storage of cache_dtype (same draw as k)
    v_cache: np.ndarray      # [T, Hkv, D] storage of cache_dtype
    heavy_tokens: List[np.ndarray] = field(default_factory=list)   # per sequence, token ids within it
    heavy_fraction: float = 0.0


def layer_inputs(w: Workload, layer: int, with_cache: bool = True) -> LayerInputs:
    """Draw one layer of the workload (deterministic in (w.base_seed, layer))."""
    g = np.random.Generator(np.random.Philox(w.base_seed + layer))
    T, Hq, Hkv, D = w.total_tokens, w.n_q_heads, w.n_kv_heads, w.head_dim
    lo, hi = w.heavy_fraction
    frac = float(lo if hi <= lo else g.uniform(lo, hi))
    q = g.standard_normal((T, Hq, D), dtype=np.float32)
    k = g.standard_normal((T, Hkv, D), dtype=np.float32)
    heavy: List[np.ndarray] = []
    cu = w.cu_seqlens
    for s, L in enumerate(w.seqlens):
        base = int(cu[s])
        n_sink = min(SINK_TOKENS, L)
        k[base:base + n_sink] *= np.float32(SINK_GAIN)
        rest = L - n_sink
        n_heavy = int(round(frac * rest)) if rest > 0 else 0
        if n_heavy > 0:
            pick = np.sort(g.choice(rest, size=n_heavy, replace=False)) + n_sink
            k[base + pick] *= np.float32(HEAVY_GAIN)
        else:
            pick = np.zeros(0, dtype=np.int64)
        heavy.append(pick.astype(np.int64))
    out_q = to_storage(q, w.qk_dtype)
    out_k = to_storage(k, w.qk_dtype)
    if with_cache:
        v = g.standard_normal((T, Hkv, D), dtype=np.float32)
        k_cache = out_k if w.cache_dtype == w.qk_dtype else to_storage(k, w.cache_dtype)
        v_cache = to_storage(v, w.cache_dtype)
    else:
        k_cache = v_cache = np.zeros((0, Hkv, D), dtype=out_k.dtype)
    return LayerInputs(out_q, out_k, k_cache, v_cache, heavy, frac)


def random_anchor_bits(n_q_heads: int, seed: int) -> np.ndarray:
    """A seeded random anchor signature: ceil(Hq/32) words, bits above Hq cleared."""
    W = (n_q_heads + 31) // 32
    g = np.random.Generator(np.random.Philox(seed))
    words = g.integers(0, 1 << 32, size=W, dtype=np.uint64).astype(np.uint32)
    tail = n_q_heads - 32 * (W - 1)
    if tail < 32:
        words[-1] &= np.uint32((1 << tail) - 1)
    return words


def random_scores(n_q_heads: int, L: int, seed: int, tie_levels: int = 0) -> np.ndarray:
    """Seeded positive float32 array [Hq, L] shaped like attention column sums.

    Used to feed the selection stages directly. ``tie_levels > 0`` quantises the
    values to that many distinct levels so that ties are frequent.
    """
    g = np.random.Generator(np.random.Philox(seed))
    x = g.gamma(0.6, 1.0, size=(n_q_heads, L))
    if L > 0:
        x[:, : min(SINK_TOKENS, L)] *= 20.0
    if tie_levels > 0:
        x = np.floor(x * tie_levels) / tie_levels
    return x.astype(np.float32)
