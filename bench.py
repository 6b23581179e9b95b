#!/usr/bin/env python
"""Benchmark of the KVCrush compression pass (score -> signature -> select -> compact).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of synthetic input (every layer of
the workload).  Prints ONE JSON line.  `value` is prompt tokens compressed per second with
the inputs resident in HBM; `e2e` is the same through host buffers (pinned host -> device
copies of Q, K and the K/V cache, device -> host copy of the kept indices and the reduced
cache inside the timed region).  `roofline` covers the dominant kernel (the tensor-core score
sweeps); `cpu_baseline` is the float64 oracle timed on this machine's host cores on a bounded
sample.  With N > 1 (torchrun) every rank runs its own replica of the workload: the pass has
no exchange step, so there is no collective on the data path (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_00022_b200 import inputs  # noqa: E402

METRIC = "prompt tokens compressed/s (score+select+compact)"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg3_llama2_32l_8k"
# dram__bytes_read + dram__bytes_write of one sweep launch per layer, from the ncu capture of the 2-layer case:
# the column-sum sweep read 286.1 MB and wrote 5.5 MB for two layers.  Scaling by the layer count over-states the
# full workload a little: the last 37 (layer, head) pairs of a launch are handed out across heads, which costs L2
# reuse, and they are 37 of 64 pairs in the capture but 37 of 1024 in the full workload.  Valid for the kernel
# source named in NCU_TRAFFIC_SOURCE only.
NCU_DRAM_BYTES_PER_LAYER_PER_SWEEP = 145.8e6
NCU_TRAFFIC_SOURCE = ("ncu capture of score_persist_kernel<128, colsum> at commit 8454247 (2 layers of the workload, scaled by the "
                      "layer count: an upper bound, see profiles/)")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------------------------
# workload arithmetic (algorithmic work, independent of how the kernels do it)
# ---------------------------------------------------------------------------------------------

def algorithmic_work(w: inputs.Workload, window: int = 0):
    """Per step (all layers).  Causal entries per head = L(L+1)/2 (rows of the observation window only when
    window > 0); 2*D flops each; two sweeps."""
    def ent(L):
        ws = L - window if 0 < window < L else 0
        return (L * (L + 1) // 2 - ws * (ws + 1) // 2) if w.causal else (L - ws) * L
    entries = sum(ent(L) for L in w.seqlens)
    flops_per_sweep = 2 * w.head_dim * entries * w.n_q_heads * w.n_layers
    b_imp, b_rep = w.budgets()
    kept = int((b_imp + b_rep).sum())
    eb = inputs.storage_itemsize(w.cache_dtype)
    compact_bytes = 2 * 2 * kept * w.n_kv_heads * w.head_dim * eb * w.n_layers        # K and V, read + write
    T, W = w.total_tokens, (w.n_q_heads + 31) // 32
    signature_bytes = (4 * w.n_q_heads + 4 * W) * T * w.n_layers
    select_bytes = (4 * w.n_q_heads + 4 * W) * T * w.n_layers + 4 * kept * w.n_layers
    return dict(score_flops=2 * flops_per_sweep, exps=2 * entries * w.n_q_heads * w.n_layers,
                compact_bytes=compact_bytes, signature_bytes=signature_bytes, select_bytes=select_bytes, kept=kept)


# ---------------------------------------------------------------------------------------------
# multi-process plumbing (one process per GPU; the data path itself has no collective)
# ---------------------------------------------------------------------------------------------

def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def max_over_ranks(value: float, device, world: int) -> float:
    """Slowest rank's time: what the whole job waits for."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_replica: int, world: int, ms_per_step: float) -> float:
    """Every rank compresses its own replica of the workload: aggregate prompt tokens per second."""
    return tokens_per_replica * world / (ms_per_step * 1e-3)


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def stop(self, t_begin: float, t_end: float):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t_begin <= t <= t_end + 0.2] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return None
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))

    def series(self):
        """(wall time, SM MHz, board W) of every sample taken so far."""
        out = []
        for t, r in self.rows:
            try:
                out.append((t, float(r[0]), float(r[2])))
            except (ValueError, IndexError):
                continue
        return out


# ---------------------------------------------------------------------------------------------
# input staging
# ---------------------------------------------------------------------------------------------

def host_inputs(w: inputs.Workload, pinned: bool):
    """All layers of the workload as host torch tensors (storage dtypes), drawn in parallel."""
    import torch
    tq = {inputs.BF16: torch.bfloat16, inputs.FP32: torch.float32}[w.qk_dtype]
    tc = {inputs.BF16: torch.bfloat16, inputs.FP16: torch.float16, inputs.FP32: torch.float32}[w.cache_dtype]
    T = w.total_tokens
    mk = dict(pin_memory=pinned)
    q = torch.empty((w.n_layers, T, w.n_q_heads, w.head_dim), dtype=tq, **mk)
    k = torch.empty((w.n_layers, T, w.n_kv_heads, w.head_dim), dtype=tq, **mk)
    kc = k if w.cache_dtype == w.qk_dtype else torch.empty((w.n_layers, T, w.n_kv_heads, w.head_dim), dtype=tc, **mk)
    vc = torch.empty((w.n_layers, T, w.n_kv_heads, w.head_dim), dtype=tc, **mk)

    def as_t(a, dt):
        t = torch.from_numpy(a.view(np.int16)) if dt == inputs.BF16 else torch.from_numpy(a)
        return t.view(torch.bfloat16) if dt == inputs.BF16 else t

    def one(layer):
        li = inputs.layer_inputs(w, layer)
        q[layer].copy_(as_t(li.q, w.qk_dtype))
        k[layer].copy_(as_t(li.k, w.qk_dtype))
        if kc is not k:
            kc[layer].copy_(as_t(li.k_cache, w.cache_dtype))
        vc[layer].copy_(as_t(li.v_cache, w.cache_dtype))

    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 8)) as ex:
        list(ex.map(one, range(w.n_layers)))
    return q, k, kc, vc


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------

def oracle_layer_pass(w: inputs.Workload, layer: int, n_heads: int = 0):
    """One pass of the float64 oracle over one layer of the workload, timed: the score step for every sequence
    (all query heads; the first ``n_heads`` only when 0 < n_heads < all), then thresholds, signatures, selection
    and compaction of every sequence on the oracle's own float32 scores (on seeded stand-in scores when only
    some heads were scored).  Returns (seconds, heads scored)."""
    from oracle import kvcrush_oracle as O
    hs = w.n_q_heads if not n_heads or n_heads >= w.n_q_heads else n_heads
    G = w.n_q_heads // w.n_kv_heads
    cu = w.cu_seqlens
    li = inputs.layer_inputs(w, layer)
    b_imp, b_rep = w.budgets()
    t0 = time.perf_counter()
    for s in range(w.n_seqs):
        a, b = int(cu[s]), int(cu[s + 1])
        if hs == w.n_q_heads:
            c, _ = O.scores(inputs.widen(li.q[a:b], w.qk_dtype), inputs.widen(li.k[a:b], w.qk_dtype), w.causal)
            s32 = O.to_scores32(c)
        else:
            # the sampled heads keep their GQA mapping: their KV heads are expanded to one per query head
            O.scores(inputs.widen(li.q[a:b, :hs], w.qk_dtype),
                     inputs.widen(li.k[a:b][:, [h // G for h in range(hs)]], w.qk_dtype), w.causal)
            s32 = inputs.random_scores(w.n_q_heads, b - a, 7 + s)
        theta = O.thresholds(s32, int(b_imp[s] + b_rep[s]))
        sig = O.signatures(s32, theta)
        idx, _ = O.select(s32, sig, int(b_imp[s]), int(b_rep[s]), w.n_kv_heads)
        O.compact(li.k_cache[a:b], idx)
        O.compact(li.v_cache[a:b], idx)
    return time.perf_counter() - t0, hs


def oracle_sample_desc(w, hs, secs, layers):
    what = "all %d heads" % w.n_q_heads if hs == w.n_q_heads else "%d of %d heads (selection on stand-in scores)" % (hs, w.n_q_heads)
    return ("oracle pass (score, thresholds, signatures, selection, compaction) over layer(s) %s of %d, %s, "
            "all %d sequence(s), %d tokens: %.2f s per layer; the step figure is that time x %d layers%s"
            % (layers, w.n_layers, what, w.n_seqs, w.total_tokens, secs, w.n_layers,
               "" if hs == w.n_q_heads else " x %d/%d heads for the score part" % (w.n_q_heads, hs)))


def cpu_baseline_leg(w: inputs.Workload):
    """The oracle as it stands on this machine's host cores: one whole layer of the workload, scaled by the layer
    count (layers are independent and of equal size)."""
    from oracle import kvcrush_oracle as O
    O.build_c()
    secs, hs = oracle_layer_pass(w, 0)
    step_s = secs * w.n_layers
    return dict(value=w.total_tokens / step_s, unit=UNIT, cores=O.n_threads(), kind="oracle",
                sample=oracle_sample_desc(w, hs, secs, "0"), extrapolation_factor=w.n_layers, sample_s=secs)


def workload_config(w: inputs.Workload, world: int, args, b_imp, b_rep):
    """The `config` object: the same keys and values from both arms."""
    eq, ec = inputs.storage_itemsize(w.qk_dtype), inputs.storage_itemsize(w.cache_dtype)
    row = w.n_layers * w.total_tokens * w.head_dim
    # Q and K for scoring, the K/V cache to compact (K serves as its own cache when the types agree)
    resident_bytes = row * (w.n_q_heads + w.n_kv_heads) * eq + row * w.n_kv_heads * ec * (1 if w.cache_dtype == w.qk_dtype else 2)
    return {"workload": w.name, "layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "n_seqs": w.n_seqs, "total_tokens": w.total_tokens,
            "budget_per_seq": [int(b_imp[0] + b_rep[0])], "cache_dtype": w.cache_dtype,
            "l2": "inputs %s L2 (%.2f GiB resident per step)" % ("larger than" if resident_bytes > 126e6 else "smaller than", resident_bytes / 2 ** 30),
            "parallelism": "replicas only" if world > 1 else "single GPU",
            "query_window": args.window, "pool_kernel": args.pool, "page_size": args.page_size,
            "keep_initial": args.keep_initial, "keep_recent": max(args.window, args.keep_recent)}




def run_reference(args, w):
    """The oracle, as it stands, on the host cores.  One step = the oracle's whole pass over ONE layer of the
    workload (step i takes layer i mod layers); `ms_per_step` is the measured time of such a step and `value`
    divides the workload's tokens by that time x the layer count (`extrapolation_factor`).  With --steps equal to
    the layer count and --warmup 0 every layer is visited once and `full_pass_s` is the whole workload, measured."""
    rank, world, _ = dist_env()
    if rank != 0:                      # under torchrun only rank 0 runs the CPU oracle; the others leave
        return
    from oracle import kvcrush_oracle as O
    O.build_c()
    threads = O.n_threads()
    b_imp, b_rep = w.budgets()
    t_run = time.perf_counter()
    # calibration (not a step): one round of heads on layer 0 tells whether whole layers fit the time budget
    cal_heads = min(w.n_q_heads, threads)
    cal_s, _ = oracle_layer_pass(w, 0, cal_heads)
    rounds = -(-w.n_q_heads // cal_heads)
    n_req = args.warmup + args.steps
    heads = 0                                              # whole layers
    steps, warmup = args.steps, args.warmup
    if cal_s * rounds * n_req > args.reference_budget_s:
        heads = cal_heads if cal_heads < w.n_q_heads else 0
        per = cal_s if heads else cal_s * rounds
        fit = max(1, int(args.reference_budget_s / per))
        if fit < n_req:                                    # still too long: fewer steps, said in the line
            warmup = min(warmup, max(0, fit - 1) // 4)
            steps = max(1, min(steps, fit - warmup))
    for i in range(warmup):
        oracle_layer_pass(w, i % w.n_layers, heads)
    secs, layers, hs = [], [], w.n_q_heads
    for i in range(steps):
        layer = (warmup + i) % w.n_layers
        t, hs = oracle_layer_pass(w, layer, heads)
        secs.append(t)
        layers.append(layer)
    mean_s = float(np.mean(secs))
    factor = w.n_layers * (w.n_q_heads / hs)
    step_s = mean_s * factor
    value = w.total_tokens / step_s
    sample = oracle_sample_desc(w, hs, mean_s, "%d..%d" % (layers[0], layers[-1]) if len(set(layers)) > 1 else str(layers[0]))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": 1e3 * mean_s, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, world, args, b_imp, b_rep),
        "extrapolation_factor": factor, "workload_ms_per_step": 1e3 * step_s,
        "steps_requested": args.steps, "warmup_requested": args.warmup,
        "note": "a step is the oracle's pass over one layer (measured); value = workload tokens / (ms_per_step x extrapolation_factor)",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "run_s": None,
    }
    if hs == w.n_q_heads and sorted(set(layers)) == list(range(w.n_layers)):
        line["full_pass_s"] = float(np.sum([np.mean([t for t, l in zip(secs, layers) if l == x]) for x in range(w.n_layers)]))
        line["full_pass_tokens_per_s"] = w.total_tokens / line["full_pass_s"]
    line["run_s"] = time.perf_counter() - t_run
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------

def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2503_00022_b200 import binding as B
    from paper_2503_00022_b200 import build as kbuild

    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        kbuild.build()
    if world > 1:
        dist.barrier()
    B.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    hq, hk, hkc, hvc = host_inputs(w, pinned=True)
    q, k = hq.to(dev, non_blocking=True), hk.to(dev, non_blocking=True)
    kc = k if hkc is hk else hkc.to(dev, non_blocking=True)
    vc = hvc.to(dev, non_blocking=True)
    tc = vc.dtype
    prob = B.Problem(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, causal=w.causal, device=dev,
                     query_window=args.window)
    b_imp, b_rep = w.budgets()
    if args.page_size:                                    # page-granular eviction: the same token budget, in whole pages
        pages = np.maximum((b_imp + b_rep) // args.page_size, 1)
        b_rep = (pages // 2).astype(np.int32)
        b_imp = (pages - b_rep).astype(np.int32)
    unit = max(args.page_size, 1)                         # decree lengths are given in tokens; pages in page mode
    keep_recent = max(args.window, args.keep_recent) // unit
    keep_initial = args.keep_initial // unit
    cp = B.CompressionPass(prob, b_imp[None, :], b_rep[None, :], cache_dtype=tc, impl=B.SCORE_AUTO,
                           pool_kernel=args.pool, keep_recent=keep_recent, page_size=args.page_size,
                           keep_initial=keep_initial)
    torch.cuda.synchronize()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]

    def step(marks=None):
        if marks: marks[0].record()
        cp.score(q, k)
        if cp.pooled is not None:
            cp.pool()
        if marks: marks[1].record()
        cp.signature()
        if marks: marks[2].record()
        cp.select()
        if marks: marks[3].record()
        cp.compact(kc, vc)
        if marks: marks[4].record()

    for _ in range(args.warmup):
        step()
    barrier()
    cp.check_status()
    sampler = ClockSampler(local) if rank == 0 else None
    t_begin = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        step(ev[i])
    e1.record()
    barrier()
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end) if sampler else None
    cp.check_status()
    total_ms = e0.elapsed_time(e1)
    stage_all = np.asarray([[ev[i][j].elapsed_time(ev[i][j + 1]) for j in range(4)] for i in range(args.steps)])
    stage_ms = stage_all.mean(axis=0)
    total_ms = max_over_ranks(total_ms, dev, world)
    ms_per_step = total_ms / args.steps

    # ---- the unchanged pass looped for several seconds: the board settles at its power limit and the SM clock it
    # sustains there, which is the condition the sustained GEMM peak was measured under ----
    sus = None
    if args.sustained_s > 0:
        n_sus = max(args.steps, int(np.ceil(args.sustained_s * 1e3 / ms_per_step)))
        ev_s = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_sus)]
        sampler_s = ClockSampler(local) if rank == 0 else None
        barrier()
        t_b = time.time()
        e0.record()
        for i in range(n_sus):
            ev_s[i][0].record()
            cp.score(q, k)
            if cp.pooled is not None:
                cp.pool()
            ev_s[i][1].record()
            cp.signature()
            cp.select()
            cp.compact(kc, vc)
        e1.record()
        barrier()
        t_e = time.time()
        clocks_s = sampler_s.stop(t_b + 1.0, t_e) if sampler_s else None      # the first second is the ramp
        cp.check_status()
        sus_ms = max_over_ranks(e0.elapsed_time(e1), dev, world) / n_sus
        half = n_sus // 2                                                     # settled part of the loop
        score_each = [a_.elapsed_time(b_) for a_, b_ in ev_s]
        sus_score_ms = float(np.mean(score_each[half:]))
        sus = dict(steps=n_sus, seconds=sus_ms * n_sus * 1e-3, ms_per_step=sus_ms, score_ms_settled=sus_score_ms,
                   clocks=clocks_s)
        # the unchanged kernels against the clock they ran at: eight windows of the loop, each with the mean score-stage
        # time of its steps, the median sampled SM clock and board power, and their product (Mcycles per step)
        if sampler_s:
            start = [e0.elapsed_time(a_) * 1e-3 for a_, _ in ev_s]            # device-time offset of every step
            ser = sampler_s.series()
            wins = []
            span = sus["seconds"]
            for i in range(8):
                lo, hi = span * i / 8, span * (i + 1) / 8
                ms_w = [m for m, t0_ in zip(score_each, start) if lo <= t0_ < hi]
                mhz_w = [mhz for t_, mhz, _ in ser if lo <= t_ - t_b < hi]
                pw_w = [pw for t_, _, pw in ser if lo <= t_ - t_b < hi]
                if ms_w and mhz_w:
                    wins.append({"t_s": round(lo, 2), "score_ms": float(np.mean(ms_w)), "sm_mhz": float(np.median(mhz_w)),
                                 "board_w": float(np.median(pw_w)), "score_ms_x_ghz": float(np.mean(ms_w) * np.median(mhz_w) * 1e-3)})
            sus["windows"] = wins

    # ---- the same pass when the caller already has the row log-sum-exp (a prefill attention kernel returns it):
    # the first sweep is skipped.  Reported beside the headline, never instead of it.
    lse_nat = cp.lse.clone()
    def step_with_lse():
        cp.score(q, k, lse_in=lse_nat)
        if cp.pooled is not None:
            cp.pool()
        cp.signature()
        cp.select()
        cp.compact(kc, vc)
    for _ in range(2):
        step_with_lse()
    barrier()
    e0.record()
    for _ in range(args.steps):
        step_with_lse()
    e1.record()
    barrier()
    lse_ms = max_over_ranks(e0.elapsed_time(e1), dev, world) / args.steps
    cp.check_status()

    # ---- signature / select / compact with a cold L2: in the pass they find the scores that sweep 2 has just written
    # in L2; here a 512 MiB buffer is overwritten before each of them
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    cold = []
    for _ in range(min(args.steps, 5)):
        row = []
        for fn in (cp.signature, cp.select, lambda: cp.compact(kc, vc)):
            flush.fill_(1)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            row.append(e0.elapsed_time(e1))
        cold.append(row)
    cold_ms = [float(x) for x in np.median(np.asarray(cold), axis=0)]
    del flush
    cp.check_status()

    # ---- the same pass recorded once into a CUDA graph and replayed (one launch per step instead of eight) ----
    cp.capture(q, k, kc, vc)
    for _ in range(2):
        cp.replay()
    barrier()
    e0.record()
    for _ in range(args.steps):
        cp.replay()
    e1.record()
    barrier()
    graph_ms = max_over_ranks(e0.elapsed_time(e1), dev, world) / args.steps
    cp.check_status()

    # ---- the clustering baseline of the paper's ablation (k-means, 100 iterations, in the place of Algorithm 2's grouping)
    # timed beside the selection stage on the same scores and signatures ----
    kmeans = None
    if args.kmeans and not args.page_size:
        K = int(b_rep.max())
        km_ws = torch.empty(max(256, B.kvcrush_kmeans_workspace_size(prob, K)), dtype=torch.uint8, device=dev)
        km_idx, km_kind = torch.empty_like(cp.idx), torch.empty_like(cp.kind)
        sc_sel = cp.pooled if cp.pooled is not None else cp.scores
        def km():
            B.kvcrush_kmeans_select(prob, sc_sel, cp.sigs, cp.budget_imp, cp.budget_rep, K, args.kmeans, cp.cu_kept,
                                    km_idx, kind=km_kind, keep_initial=keep_initial, keep_recent=keep_recent,
                                    workspace=km_ws, status=cp.status)
        km()
        torch.cuda.synchronize()
        cp.check_status()
        reps = max(1, min(args.steps, 3))
        e0.record()
        for _ in range(reps):
            km()
        e1.record()
        torch.cuda.synchronize()
        km_ms = e0.elapsed_time(e1) / reps
        kmeans = {"iterations": args.kmeans, "ms": km_ms, "select_ms": float(stage_ms[2]), "ratio_to_select": km_ms / float(stage_ms[2]),
                  "ratio_to_whole_pass": km_ms / ms_per_step,
                  "agreement_with_kvcrush": float((torch.isin(km_idx, cp.idx).float().mean()).item()) if w.n_layers * w.n_seqs == 1 else None,
                  "note": "k-means over the same binary head vectors, k = B_representative clusters per (layer, sequence)"}
        del km_ws

    # ---- end to end through host buffers: H2D of the step's inputs, D2H of the kept set and reduced cache ----
    # Layers are independent, so the pass runs in chunks of layers: chunk c+1 is copied in (one stream) while
    # chunk c is compressed (the timed stream) and chunk c-1's kept indices and reduced cache are copied out
    # (a third stream).  Every byte still crosses the bus inside the timed region.
    e2e_steps = max(1, min(args.steps, 3))
    n_chunks = min(8, w.n_layers)
    bounds = [round(i * w.n_layers / n_chunks) for i in range(n_chunks + 1)]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream()
    passes, host_out = [], []
    for i in range(2):                                        # two sets of chunk buffers, used alternately
        nl = max(bounds[c + 1] - bounds[c] for c in range(n_chunks))
        pr = B.Problem(nl, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seqlens, causal=w.causal, device=dev,
                       query_window=args.window)
        passes.append(B.CompressionPass(pr, b_imp[None, :], b_rep[None, :], cache_dtype=tc, impl=B.SCORE_AUTO,
                                        pool_kernel=args.pool, keep_recent=keep_recent, page_size=args.page_size,
                                        keep_initial=keep_initial))
    equal_chunks = all(bounds[c + 1] - bounds[c] == bounds[1] - bounds[0] for c in range(n_chunks))
    h_idx = [torch.empty(passes[0].idx.shape, dtype=torch.int32, pin_memory=True) for _ in range(n_chunks)]
    h_ko = [torch.empty(passes[0].k_out.shape, dtype=tc, pin_memory=True) for _ in range(n_chunks)]
    h_vo = [torch.empty(passes[0].v_out.shape, dtype=tc, pin_memory=True) for _ in range(n_chunks)]

    def e2e_step():
        ev_in = [torch.cuda.Event() for _ in range(n_chunks)]
        ev_done = [torch.cuda.Event() for _ in range(n_chunks)]
        ev_out = [torch.cuda.Event() for _ in range(n_chunks)]
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        for c in range(n_chunks):
            a_, b_ = bounds[c], bounds[c + 1]
            with torch.cuda.stream(s_in):
                q[a_:b_].copy_(hq[a_:b_], non_blocking=True)
                k[a_:b_].copy_(hk[a_:b_], non_blocking=True)
                if kc is not k:
                    kc[a_:b_].copy_(hkc[a_:b_], non_blocking=True)
                vc[a_:b_].copy_(hvc[a_:b_], non_blocking=True)
                ev_in[c].record(s_in)
            pc = passes[c & 1]
            main.wait_event(ev_in[c])
            if c >= 2:
                main.wait_event(ev_out[c - 2])                # this buffer set's previous results have left
            pc.run(q[a_:b_], k[a_:b_], kc[a_:b_], vc[a_:b_])
            ev_done[c].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[c])
                h_idx[c].copy_(pc.idx, non_blocking=True)
                h_ko[c].copy_(pc.k_out, non_blocking=True)
                h_vo[c].copy_(pc.v_out, non_blocking=True)
                ev_out[c].record(s_out)
        main.wait_stream(s_out)

    if not equal_chunks:                                      # uneven chunks would not fit the shared chunk problem
        n_chunks, bounds = 1, [0, w.n_layers]
        passes = [cp, cp]
        h_idx, h_ko, h_vo = ([torch.empty(t.shape, dtype=t.dtype, pin_memory=True)] for t in (cp.idx, cp.k_out, cp.v_out))
    e2e_step()
    barrier()
    for pc in passes:
        pc.check_status()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, dev, world) / e2e_steps
    nbytes = lambda t: t.numel() * t.element_size()  # noqa: E731
    h2d = nbytes(hq) + nbytes(hk) + (nbytes(hkc) if hkc is not hk else 0) + nbytes(hvc)
    d2h = sum(nbytes(t) for t in h_idx + h_ko + h_vo)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    work = algorithmic_work(w, args.window)
    if args.page_size:                                    # rows actually gathered: kept pages x page size
        eb = inputs.storage_itemsize(w.cache_dtype)
        work["compact_bytes"] = 2 * 2 * cp.total_kept * args.page_size * w.n_kv_heads * w.head_dim * eb
    score_s = stage_ms[0] * 1e-3
    tensor_path = cp.impl != B.SCORE_SIMT and w.qk_dtype in (inputs.BF16, inputs.FP16) and w.head_dim % 8 == 0 and w.head_dim <= 128
    short_tf = work["score_flops"] / score_s / 1e12
    if tensor_path:
        # Headline fraction: the score stage inside the seconds-long loop against the sustained GEMM peak (both at the
        # board's power limit); beside it the K-step loop against the burst peak (both short).
        sus_tf = work["score_flops"] / (sus["score_ms_settled"] * 1e-3) / 1e12 if sus else short_tf
        launch_ms = (sus["score_ms_settled"] if sus else float(stage_ms[0])) / 2
        whole = w.name == DEFAULT_WORKLOAD or w.name.startswith(DEFAULT_WORKLOAD + "_")
        traffic = NCU_DRAM_BYTES_PER_LAYER_PER_SWEEP * w.n_layers if (whole and not args.window) else None
        roofline = {"bound": "tensor", "kernel": "score_persist_kernel (two sweep launches per step; per-launch figures)",
                    "achieved": sus_tf, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                    "frac": sus_tf / peaks["bf16_tflops_sustained"],
                    "timing": ("score stage, CUDA events, settled half of a %.1f s loop of the whole pass" % sus["seconds"]) if sus else "score stage of the timed steps",
                    "peak_source": peaks["source"] + " (sustained bf16: seconds-long loop under the power cap)",
                    "traffic": traffic, "traffic_source": NCU_TRAFFIC_SOURCE if traffic else None,
                    "algorithmic_flops_per_launch": work["score_flops"] / 2, "launch_ms": launch_ms,
                    "short_loop": {"achieved": short_tf, "peak": peaks["bf16_tflops"], "frac": short_tf / peaks["bf16_tflops"],
                                   "launch_ms": float(stage_ms[0]) / 2,
                                   "note": "score stage of the %d timed steps against the burst bf16 peak" % args.steps},
                    "frac_of_nominal_2250": sus_tf / 2250.0,
                    "exps_per_s": work["exps"] / (2 * launch_ms * 1e-3)}
        if sus and sus["clocks"]:
            ghz = sus["clocks"]["sm_mhz"] * 1e-3
            roofline["sm_ghz_sustained"] = ghz
            roofline["launch_ms_x_ghz"] = launch_ms * ghz          # clock-independent cost of one sweep: Mcycles
            # context: the other unit the sweeps load - one exponential per causal logit per sweep, 16 per clock per SM
            # on the special-function unit at the sampled clock (a quarter of them are evaluated on the FMA pipe instead)
            n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
            sfu_peak = n_sm * 16 * ghz * 1e9
            roofline["exp_unit"] = {"exps_per_s": roofline["exps_per_s"], "sfu_peak_per_s": sfu_peak,
                                    "frac_if_all_on_sfu": roofline["exps_per_s"] / sfu_peak,
                                    "sfu_share_of_exps": 0.75}
    else:
        # fp32 FMA on the CUDA cores: 128 lanes x 2 flop per SM per clock at the SM clock sampled during the timed steps
        n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = clocks["sm_mhz"] if clocks else 1965.0
        peak_tf = n_sm * 128 * 2 * mhz * 1e6 / 1e12
        roofline = {"bound": "alu", "kernel": "score SIMT kernels (fp32 FMA on the CUDA cores)", "achieved": short_tf,
                    "peak": peak_tf, "unit": "TFLOP/s", "frac": short_tf / peak_tf, "traffic": None,
                    "peak_source": "derived: %d SMs x 128 fp32 lanes x 2 flop x %.0f MHz (sampled SM clock)" % (n_sm, mhz),
                    "algorithmic_flops_per_launch": work["score_flops"] / 2, "launch_ms": float(stage_ms[0]) / 2}
    hbm = peaks["hbm_gbs"]
    stages = {
        "score_ms": float(stage_ms[0]), "signature_ms": float(stage_ms[1]), "select_ms": float(stage_ms[2]),
        "compact_ms": float(stage_ms[3]),
        "compact_gbs": work["compact_bytes"] / (stage_ms[3] * 1e-3) / 1e9,
        "compact_frac_hbm": work["compact_bytes"] / (stage_ms[3] * 1e-3) / 1e9 / hbm,
        "signature_gbs": work["signature_bytes"] / (stage_ms[1] * 1e-3) / 1e9,
        "select_gbs": work["select_bytes"] / (stage_ms[2] * 1e-3) / 1e9,
        "hbm_peak_gbs": hbm, "hbm_peak_source": peaks["source"],
        "median_ms": [float(x) for x in np.median(stage_all, axis=0)], "min_ms": [float(x) for x in stage_all.min(axis=0)],
        "order": ["score", "signature", "select", "compact"],
        "graph_replay_ms_per_step": graph_ms,
        "cold_l2_ms": {"signature": cold_ms[0], "select": cold_ms[1], "compact": cold_ms[2],
                       "note": "512 MiB overwritten before each stage; medians"},
    }
    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline_leg(w)

    tokens = w.total_tokens * world
    # kernels of this library per step: two score sweeps, threshold select + signature pack (which also writes the token
    # importance), the segment selection, the gather (+ pooling)
    launches_per_step = 2 + 2 + (1 if cp.importance is not None else 2) + 1 + (1 if cp.pooled is not None else 0)
    line = {
        "metric": METRIC, "value": whole_job_value(w.total_tokens, world, ms_per_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.qk_dtype == inputs.BF16 else "f32", "data": "synthetic",
        "config": workload_config(w, world, args, b_imp, b_rep),
        "layer_tokens_per_s": tokens * w.n_layers / (ms_per_step * 1e-3),
        "roofline": roofline, "stages": stages, "cpu_baseline": cpu,
        "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": e2e_ms, "layer_chunks": n_chunks,
                "overlap": "H2D, compute and D2H of consecutive layer chunks on three streams"},
        "lse_supplied": {"ms_per_step": lse_ms, "value": whole_job_value(w.total_tokens, world, lse_ms), "unit": UNIT,
                         "note": "row log-sum-exp given by the caller: one score sweep instead of two"},
        "sustained": sus, "kmeans_baseline": kmeans,
        "gpu_launches": launches_per_step * args.steps,
        "gpu_launches_per_step": launches_per_step,
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--layers", type=int, default=0, help="run only this many layers of the workload (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--reference-budget-s", type=float, default=450.0,
                    help="--impl reference: the run (warm-up + steps) is sized to end within this many seconds; a whole pass "
                         "of the oracle over every layer (--steps LAYERS --warmup 0) needs more")
    ap.add_argument("--kmeans", type=int, default=0,
                    help="also time the k-means clustering baseline with this many iterations (the paper's ablation uses 100)")
    ap.add_argument("--sustained-s", type=float, default=4.0,
                    help="also loop the pass for at least this many seconds (0 = skip); the roofline fraction is taken there")
    ap.add_argument("--window", type=int, default=0,
                    help="SnapKV-style importance: only the last WINDOW queries vote and those tokens are kept (0 = H2O, all queries)")
    ap.add_argument("--pool", type=int, default=0, help="max-pool the per-head scores with this odd kernel width (0 = off)")
    ap.add_argument("--page-size", type=int, default=0,
                    help="evict whole pages of this many tokens (8 = the paper's chunks, 32 = its pages; 0 = token level)")
    ap.add_argument("--keep-initial", type=int, default=0, help="first tokens of every sequence kept by decree (attention sinks)")
    ap.add_argument("--keep-recent", type=int, default=0, help="last tokens of every sequence kept by decree")
    args = ap.parse_args()
    if args.page_size and args.window:
        ap.error("--page-size and --window are separate modes")
    w = inputs.paper_workloads()[args.workload]
    if args.layers:
        w = inputs.shrink(w, args.layers)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
