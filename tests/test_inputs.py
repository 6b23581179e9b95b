"""The seeded workload generator: determinism, storage rounding, structure."""
import numpy as np
import torch

from paper_2503_00022_b200 import inputs


def test_bf16_rounding_matches_torch():
    g = np.random.Generator(np.random.Philox(3))
    x = (g.standard_normal(20000) * np.exp(g.uniform(-20, 20, 20000))).astype(np.float32)
    bits = inputs.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    back = inputs.bf16_bits_to_f32(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_layer_inputs_are_deterministic_and_structured():
    w = inputs.Workload("t", 2, 4, 2, 16, (40, 300), inputs.BF16, inputs.FP16, 0.25, base_seed=9)
    a = inputs.layer_inputs(w, 1)
    b = inputs.layer_inputs(w, 1)
    c = inputs.layer_inputs(w, 0)
    assert a.q.tobytes() == b.q.tobytes() and a.k.tobytes() == b.k.tobytes()
    assert a.v_cache.tobytes() == b.v_cache.tobytes()
    assert a.q.tobytes() != c.q.tobytes()
    assert a.q.shape == (340, 4, 16) and a.k.shape == (340, 2, 16) and a.q.dtype == np.uint16
    assert a.k_cache.dtype == np.float16 and a.v_cache.shape == (340, 2, 16)
    k = inputs.widen(a.k, w.qk_dtype)
    norms = np.sqrt((k ** 2).sum(axis=(1, 2)))
    cu = w.cu_seqlens
    for s, L in enumerate(w.seqlens):
        seg = norms[cu[s]:cu[s + 1]]
        plain = np.ones(L, dtype=bool)
        plain[:4] = False
        plain[a.heavy_tokens[s]] = False
        assert len(a.heavy_tokens[s]) == round(0.05 * (L - 4))
        assert seg[:4].mean() > 3.0 * seg[plain].mean()
        if len(a.heavy_tokens[s]):
            assert seg[a.heavy_tokens[s]].mean() > 1.6 * seg[plain].mean()


def test_paper_workloads_shapes_and_budgets():
    ws = inputs.paper_workloads()
    assert [w.total_tokens for w in ws.values()][:4] == [512, 4096, 8192, 32768]
    imp, rep = ws["cfg4_llama3_gqa_32k"].budgets()
    assert (int(imp[0]), int(rep[0])) == (3277, 3277)
    w5 = ws["cfg5_ragged_batch16"]
    assert w5.n_seqs == 16 and all(1024 <= L <= 4096 for L in w5.seqlens)
    imp, rep = w5.budgets()
    for L, i, r in zip(w5.seqlens, imp, rep):
        assert i + r == L // 4 and r == (L // 4) // 2
    assert w5.cu_seqlens[-1] == w5.total_tokens
    lo, hi = ws["cfg3_llama2_32l_8k"].heavy_fraction
    fr = [inputs.layer_inputs(inputs.Workload("x", 4, 1, 1, 8, (64,), inputs.BF16, inputs.BF16, 0.25,
                                               heavy_fraction=(lo, hi), base_seed=1300), l, False).heavy_fraction
          for l in range(4)]
    assert all(lo <= f <= hi for f in fr) and len(set(fr)) == 4
