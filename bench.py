#!/usr/bin/env python
"""Benchmark of the measure -> recover -> execute FFN step.

A step is one pass of the whole path (sketch, recovery, sparse FFN) over one decode batch of a
synthetic layer (one prompt through one layer for the prompt-level variant).  The headline workload
is the Llama-2-7B-shaped layer at decode batch 1; the other workloads (batch 64, the 32-layer stack,
the prompt-level variant at three sparsity levels, the tiny f32 case) are timed in the same run and
reported under "workloads".  Steps rotate over several distinct layers and token batches (more weight
bytes than the L2 holds), so every step streams its active rows from HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Timing: W untimed warm-up steps, extended until at least 0.2 s of device work has run (a GPU that was
idle takes that long to reach its clocks); then the region of exactly K steps, bracketed by a
barrier and a device synchronisation on both sides and timed with CUDA events on the launching
stream, is repeated until at least 0.5 s have been timed.  The reported step time is the median over
the repeats (maximum over ranks of every repeat).  Clocks are sampled over the whole timed span.

Under torchrun (N > 1) every rank runs the same per-GPU workload on its own tokens (weak scaling,
no collective on the data path).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from gen import workloads as W  # noqa: E402
from paper_2604_14156_b200 import shard  # noqa: E402

METRIC = "sparse_ffn_decode_tokens_per_s_per_layer"
UNIT = "tokens/s"
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the roofline kernels, from the
# ncu captures summarised under profiles/, keyed by (workload, k).  An entry is removed when its
# kernel changes and comes back with the next capture; a missing entry reports null.
NCU_TRAFFIC = {
    ("l2_7b_b1", 22): 69.24e6 + 1.34e6,                       # ffn_gather_kernel
    ("l2_7b_b64", 22): 181.44e6 + 3.52e6 + 95.85e6 + 3.53e6,  # ffn_gateup_swap_kernel + ffn_down_swap_kernel
    ("l2_13b_prompt", 27): 211.12e6 + 12.08e6 + 56.08e6 + 5.21e6,  # ffn_gateup_pair_kernel + ffn_down_wide_kernel
}
GRAPH_STEPS = 64          # most steps captured per CUDA graph
N_TOKEN_BATCHES = 16      # distinct input batches rotated through
WARM_SECONDS = 0.2
TIMED_SECONDS = 0.5
MAX_REPEATS = 5000
EXTRA_WORKLOADS = ["l2_7b_b64", "l3_8b_stack", "l2_13b_prompt:11", "l2_13b_prompt:27", "l2_13b_prompt:54", "tiny_f32"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="l2_7b_b1",
                    choices=["l2_7b_b1", "l2_7b_b64", "l3_8b_stack", "tiny_f32", "l2_13b_prompt"])
    ap.add_argument("--k", type=int, default=0, help="active groups (prompt workload sweep: 11 / 27 / 54)")
    ap.add_argument("--layers", type=int, default=0, help="distinct layers rotated through (0 = auto)")
    ap.add_argument("--batch", type=int, default=0, help="decode batch override (regime sweeps; 0 = the workload's own)")
    ap.add_argument("--crossover", type=int, default=0,
                    help="smallest batch that takes the tensor-core path (regime sweeps; 0 = the plan's own)")
    ap.add_argument("--no-extra", action="store_true", help="time the named workload only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, 'measured' | 'fallback')."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops_sustained", p.get("bf16_tflops", 1400.0))), "measured"
    return 6650.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.period = period_s

    def _run(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_min_mhz": s[0] if s else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}


class Timer:
    """Times a region of K steps on `stream` as the docstring of this file says."""

    def __init__(self, stream, dev, world):
        self.stream, self.dev, self.world = stream, dev, world

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()

    def once(self, run, n) -> float:
        """Milliseconds of run(n): barrier + synchronise, event, run, event, synchronise + barrier; max over ranks."""
        self.barrier(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        run(n)
        e1.record(self.stream)
        torch.cuda.synchronize(); self.barrier()
        return shard.max_over_ranks(e0.elapsed_time(e1), self.dev)

    def measure(self, run, K, warmup, warm_s=WARM_SECONDS, timed_s=TIMED_SECONDS):
        """(median ms of a K-step region, repeats, all region times) after the warm-up."""
        run(warmup)
        torch.cuda.synchronize()
        spent = 0.0
        while spent < warm_s * 1e3:
            spent += max(self.once(run, K), 1e-3)
        est = self.once(run, K)
        repeats = int(min(MAX_REPEATS, max(3, math.ceil(timed_s * 1e3 / max(est, 1e-3)))))
        times = [self.once(run, K) for _ in range(repeats)]
        return statistics.median(times), repeats, times


def algorithmic_bytes(cfg: W.Config, union_groups: float) -> dict:
    """Bytes the method itself must move per step: active weight blocks (union over the batch,
    counted once), the sketch matrix, Phi, and the activations in and out."""
    wbytes = 2 if cfg.w_dtype == "bf16" else 4
    weights = 3 * union_groups * cfg.group * cfg.d * wbytes
    sketch = cfg.m * cfg.d * 4 + cfg.m * cfg.G * 4
    act = 2 * cfg.B * cfg.d * 4
    return {"weights": weights, "sketch": sketch, "activations": act, "total": weights + sketch + act}


def graph_runner(step, chunk, stream):
    """Captures `chunk` consecutive steps into a CUDA graph; returns run(n) for n a multiple of chunk
    (a remainder is launched step by step)."""
    for i in range(3):
        step(i)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for i in range(chunk):
            step(i)

    def run(n):
        for _ in range(n // chunk):
            graph.replay()
        for i in range(n % chunk):
            step(i)
    return run, graph


def bench_decode(cfg, args, K, Wm, rank, world, local, dev, primary):
    """One decode workload; returns the result dictionary (the JSON line's keys for the primary)."""
    import paper_2604_14156_b200 as cs

    wbytes_layer = 3 * cfg.d_ff * cfg.d * (2 if cfg.w_dtype == "bf16" else 4)
    n_layers = args.layers or (cfg.n_layers if cfg.n_layers > 1 else max(4, min(16, int(4e9 // wbytes_layer))))
    n_layers = min(n_layers, GRAPH_STEPS)
    plan = cs.Plan(cfg.d, cfg.d_ff, cfg.group, cfg.m, cfg.k, cfg.T,
                   torch.float32 if cfg.w_dtype == "f32" else torch.bfloat16, cfg.B, cfg.rms_eps)
    if args.crossover:
        plan.set_crossover(args.crossover)
    layers_raw, layers = [], []
    for i in range(n_layers):
        L = W.make_layer(cfg, i, device=dev)
        layers_raw.append(L)
        layers.append(cs.Layer(plan, L.S, L.Phi, L.W_gate, L.W_up, L.Wd_t, L.mu, L.gamma, cfg.rms))
    # each rank decodes its own tokens (weak scaling): the batch index is offset by the rank
    xs = torch.stack([W.make_tokens(cfg, layers_raw[0].A, batch=shard.batch_stream(rank, j, N_TOKEN_BATCHES)).h
                      for j in range(N_TOKEN_BATCHES)]).to(dev)
    x_out = torch.empty_like(xs[0])
    chained = cfg.n_layers > 1   # the stack: each layer's input is the previous layer's output
    x_chain = xs[0].clone()

    def step(i):
        if chained:
            cs.cs_layer_step(plan, layers[i % n_layers], x_chain, x_out=x_chain, want_aux=False)
        else:
            cs.cs_layer_step(plan, layers[i % n_layers], xs[i % N_TOKEN_BATCHES], x_out=x_out, want_aux=False)

    stream = torch.cuda.Stream(device=dev)
    timer = Timer(stream, dev, world)
    chunk = min(K, GRAPH_STEPS)
    with torch.cuda.stream(stream):
        before = plan.launches
        run_steps, _g = graph_runner(step, chunk, stream)
        launches_per_step = (plan.launches - before) / (chunk + 3)
        with ClockSampler(local) as clocks:
            ms_region, repeats, times = timer.measure(run_steps, K, Wm)

        # ---- end to end: host buffers in, host result out, through the C boundary
        hx = torch.stack([x.cpu() for x in xs]).pin_memory()
        hout = torch.empty_like(hx[0]).pin_memory()

        def step_host(i):
            cs.cs_layer_step_host(plan, layers[i % n_layers], hx[i % N_TOKEN_BATCHES], hout)

        run_host, _gh = graph_runner(step_host, chunk, stream)
        ms_e2e, _, _ = timer.measure(run_host, K, min(Wm, chunk), warm_s=0.05)

        # ---- per-stage device times: a separate pass with events around every stage's launches.  Each
        # step is replayed from a one-step CUDA graph, in which the records are event nodes: a record
        # issued from the host between two launches would add several microseconds to every bracket.
        plan.enable_timing(True)
        n_prof = 100
        n_graphs = min(n_layers * (1 if chained else 2), 32)
        stage_graphs = []
        for i in range(n_graphs):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                step(i)
            stage_graphs.append(g)
        acc = [0.0] * 5
        for i in range(n_prof + 3):
            stage_graphs[i % n_graphs].replay()
            t = plan.stage_times(stream)
            if i >= 3:
                acc = [a + b for a, b in zip(acc, t)]
        plan.enable_timing(False)
        stage_ms = [a / n_prof for a in acc]
        # union of supports of one representative batch (for the algorithmic byte count)
        _, sup_probe, _, _ = cs.cs_layer_step(plan, layers[0], xs[0])
        stream.synchronize()

        # ---- the actuator alone: the same steps with the supports given (cs_ffn_exec on the supports of
        # a finished step), timed like the step itself.  This is the duration the roofline uses, and
        # what sketch + recovery add to the step is the difference of the two figures.
        def exec_only(i):
            cs.cs_ffn_exec(plan, layers[i % n_layers], xs[i % N_TOKEN_BATCHES], sup_probe, out=x_out)

        run_exec, _gx = graph_runner(exec_only, chunk, stream)
        ms_exec, _, _ = timer.measure(run_exec, K, min(Wm, chunk), warm_s=0.05, timed_s=0.25)

    union = float(len(torch.unique(sup_probe)))
    step_us = ms_region * 1e3 / K
    exec_only_us = ms_exec * 1e3 / K
    tokens_per_s = cfg.B * world / (step_us * 1e-6)
    ab = algorithmic_bytes(cfg, union)
    peak, _, peak_kind = peaks()
    mma = cfg.B >= plan.crossover and cfg.B <= 128 and cfg.w_dtype == "bf16" and cfg.group == 128 and cfg.d % 256 == 0
    big = cfg.B > 128 and cfg.w_dtype == "bf16" and cfg.group == 128 and cfg.d % 256 == 0
    # the actuator reads the active weights and the hidden state and writes the output
    kernel_bytes = ab["weights"] + cfg.B * cfg.d * 4 * 2
    achieved = kernel_bytes / (exec_only_us * 1e-6) / 1e9
    mr_us = (stage_ms[0] + stage_ms[1]) * 1e3
    zero_copy = cfg.B * cfg.d * 4 <= (4 << 20 if (mma or big) else 64 << 10)
    out = {
        "metric": METRIC, "value": tokens_per_s, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "repeats": repeats, "ms_per_step": ms_region / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "d": cfg.d, "d_ff": cfg.d_ff, "groups": cfg.G, "group": cfg.group,
                   "m": cfg.m, "k": cfg.k, "T": cfg.T, "batch": cfg.B, "weights": cfg.w_dtype,
                   "accumulate": "f32", "layers_rotated": n_layers, "token_batches_rotated": N_TOKEN_BATCHES,
                   "l2": (f"inputs larger than L2: {n_layers} layers x {wbytes_layer / 1e6:.0f} MB rotated"
                          if n_layers * wbytes_layer > 400e6 else
                          f"L2-resident ({n_layers} layers x {wbytes_layer / 1e6:.1f} MB): a correctness workload, launch-latency bound"),
                   "cuda_graph_steps": chunk, "parallelism": f"dp{world}" if world > 1 else "single",
                   "timing": f"median of {repeats} repeats of the {K}-step region after >= {WARM_SECONDS} s of warm-up",
                   "e2e_path": ("cs_layer_step_host on pinned host buffers: x fetched over the bus by a staging kernel, "
                                "result stored into the host buffer by the step's last kernel" if zero_copy else
                                "cs_layer_step_host on pinned host buffers: copy-engine transfers around the step")},
        "e2e": {"value": cfg.B * world * K / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": cfg.B * cfg.d * 4,
                "d2h_bytes_per_step": cfg.B * cfg.d * 4},
        "gpu_launches": int(round(launches_per_step * K)),
        "clocks": clocks.summary(),
        "region_ms": {"median": ms_region, "min": min(times), "max": max(times)},
        "roofline": {"bound": "hbm",
                     "kernel": ("ffn_gateup_swap_kernel + ffn_down_swap_kernel" if mma else
                                "ffn_gateup_mma_kernel + ffn_down_mma_kernel" if big else "ffn_gather_kernel"),
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "frac_of_8tbs_nominal": achieved / 8000.0,
                     "bytes_per_launch": kernel_bytes, "avg_launch_us": exec_only_us,
                     "duration_from": ("cs_ffn_exec on given supports, graph-captured and timed like the step (CUDA events, "
                                       "median of repeats): the execution kernels plus the support check and the "
                                       "partial-sum reduction around them, so an upper bound of the kernels' own time"),
                     "bracket_us": (stage_ms[2] + stage_ms[4]) * 1e3,
                     "traffic": NCU_TRAFFIC.get((cfg.name, cfg.k)) if cfg.B == W.CONFIGS[cfg.name].B else None},
        "stages_us": {"sketch": stage_ms[0] * 1e3, "recover": stage_ms[1] * 1e3, "exec": stage_ms[2] * 1e3,
                      "exec_down": stage_ms[4] * 1e3, "reduce": stage_ms[3] * 1e3, "step_net": step_us,
                      "note": "stage figures are event brackets inside one-step graphs (2-4 us of record overhead each)",
                      "measure_recover_per_token": mr_us / cfg.B,
                      "measure_recover_share_of_step": mr_us / step_us if step_us > 0 else None,
                      "exec_only_step": exec_only_us,
                      # what sketch + recovery leave on the critical path: net step minus the actuator alone
                      "measure_recover_exposed_us": max(0.0, step_us - exec_only_us),
                      "measure_recover_exposed_share": max(0.0, step_us - exec_only_us) / step_us},
        "step_hbm": {"algorithmic_bytes": ab["total"], "gbs": ab["total"] / (step_us * 1e-6) / 1e9,
                     "frac_of_measured_peak": ab["total"] / (step_us * 1e-6) / 1e9 / peak,
                     "frac_of_8tbs_nominal": ab["total"] / (step_us * 1e-6) / 1e9 / 8000.0,
                     "union_groups": union, "groups_streamed": (cfg.G if mma else union)},
    }
    if primary and rank == 0:
        out["planted_recovery"] = planted_recovery(cfg, dev)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_layers = [L.to("cpu") for L in layers_raw[:2]]
        out["cpu_baseline"] = cpu_baseline(cfg, cpu_layers, hx, seconds=10.0 if primary else 3.0, single=primary)
    plan.close()
    return out


def bench_prompt(cfg, args, K, Wm, rank, world, local, dev, primary):
    """Prompt-level variant: one support from the mean prompt sketch, then the FFN of all 2048 prompt
    tokens over that support as grouped GEMMs.  A step is one prompt through one layer."""
    import paper_2604_14156_b200 as cs
    n_layers = args.layers or 8
    plan = cs.Plan(cfg.d, cfg.d_ff, cfg.group, cfg.m, cfg.k, cfg.T, torch.bfloat16, cfg.B, cfg.rms_eps)
    raw = [W.make_layer(cfg, i, device=dev) for i in range(n_layers)]
    layers = [cs.Layer(plan, L.S, L.Phi, L.W_gate, L.W_up, L.Wd_t, L.mu) for L in raw]
    Hs = torch.stack([W.make_tokens(cfg, raw[0].A, batch=rank * 4 + j).h for j in range(4)]).to(dev)
    out = torch.empty_like(Hs[0])
    stream = torch.cuda.Stream(device=dev)
    timer = Timer(stream, dev, world)

    def step(i):
        L = raw[i % n_layers]
        s, _, _ = cs.cs_prompt_support(plan, L.S, L.Phi, L.mu, Hs[i % 4])
        cs.cs_ffn_exec_shared(plan, layers[i % n_layers], Hs[i % 4], s, out=out)

    def run(n):
        for i in range(n):
            step(i)

    with torch.cuda.stream(stream):
        run(3); stream.synchronize()
        before = plan.launches
        run(K)
        launches = plan.launches - before
        with ClockSampler(local) as clocks:
            ms_region, repeats, times = timer.measure(run, K, Wm)
        hH = Hs.cpu().pin_memory(); hout = torch.empty_like(hH[0]).pin_memory()
        Hd = torch.empty_like(Hs[0])

        def run_host(n):
            for i in range(n):
                Hd.copy_(hH[i % 4], non_blocking=True)
                L = raw[i % n_layers]
                s, _, _ = cs.cs_prompt_support(plan, L.S, L.Phi, L.mu, Hd)
                cs.cs_ffn_exec_shared(plan, layers[i % n_layers], Hd, s, out=out)
                hout.copy_(out, non_blocking=True)

        ms_e2e, _, _ = timer.measure(run_host, K, 3, warm_s=0.05, timed_s=0.25)
        # the two grouped GEMMs alone, on a given support
        sup, _, _ = cs.cs_prompt_support(plan, raw[0].S, raw[0].Phi, raw[0].mu, Hs[0])
        stream.synchronize()

        def run_exec(n):
            for i in range(n):
                cs.cs_ffn_exec_shared(plan, layers[i % n_layers], Hs[i % 4], sup, out=out)

        ms_exec, _, _ = timer.measure(run_exec, K, 3, warm_s=0.05, timed_s=0.25)
        plan.enable_timing(True)
        acc = [0.0] * 5
        n_prof = 20
        for i in range(n_prof + 3):
            step(i)
            t = plan.stage_times(stream)
            if i >= 3:
                acc = [a + b for a, b in zip(acc, t)]
        plan.enable_timing(False)
    stage_ms = [a / n_prof for a in acc]
    _, tf_peak, kind = peaks()
    flops = 6.0 * cfg.B * cfg.k * cfg.group * cfg.d
    exec_us = ms_exec * 1e3 / K
    achieved = flops / (exec_us * 1e-6) / 1e12
    step_us = ms_region * 1e3 / K
    res = {
        "metric": METRIC, "value": cfg.B * world / (step_us * 1e-6), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": Wm, "repeats": repeats, "ms_per_step": ms_region / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "d": cfg.d, "d_ff": cfg.d_ff, "groups": cfg.G, "group": cfg.group,
                   "m": cfg.m, "k": cfg.k, "T": cfg.T, "prompt_tokens": cfg.B, "weights": "bf16",
                   "accumulate": "f32", "layers_rotated": n_layers,
                   "l2": f"inputs larger than L2: {n_layers} layers rotated, 4 prompts of {cfg.B * cfg.d * 2 / 1e6:.0f} MB",
                   "timing": f"median of {repeats} repeats of the {K}-step region after >= {WARM_SECONDS} s of warm-up",
                   "e2e_path": "pinned host copies around the device entry points",
                   "parallelism": f"dp{world}" if world > 1 else "single"},
        "e2e": {"value": cfg.B * world * K / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": cfg.B * cfg.d * 2,
                "d2h_bytes_per_step": cfg.B * cfg.d * 2},
        "gpu_launches": launches, "clocks": clocks.summary(),
        "region_ms": {"median": ms_region, "min": min(times), "max": max(times)},
        "roofline": {"bound": "tensor", "kernel": "ffn_gateup_tiles_kernel (paired token tiles where they shorten the last wave; else ffn_gateup_pair_kernel, CTA pairs with M = 256) + ffn_down_wide_kernel (ffn_down_mma_kernel where it needs fewer rounds)",
                     "achieved": achieved, "peak": tf_peak, "unit": "TFLOP/s", "frac": achieved / tf_peak,
                     "peak_kind": kind + " (sustained)", "flops_per_launch_pair": flops, "avg_pair_us": exec_us,
                     "duration_from": "cs_ffn_exec_shared on a given support, timed like the step (CUDA events, median of repeats)",
                     "bracket_us": stage_ms[2] * 1e3,
                     "traffic": NCU_TRAFFIC.get((cfg.name, cfg.k))},
        "stages_us": {"mean_sketch": stage_ms[0] * 1e3, "recover": stage_ms[1] * 1e3, "exec": stage_ms[2] * 1e3,
                      "reduce": stage_ms[3] * 1e3, "step_net": step_us, "exec_only_step": exec_us,
                      "measure_recover_exposed_share": max(0.0, step_us - exec_us) / step_us},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        res["cpu_baseline"] = cpu_baseline_prompt(cfg, raw[0].to("cpu"), Hs[0].cpu(), seconds=10.0 if primary else 3.0)
    plan.close()
    return res


def planted_recovery(cfg, dev, trials: int = 256):
    """How often each estimator returns a planted support (noiseless, |c| >= 0.5) at this workload's m and G,
    for sparsity levels from easy to the workload's own k: the library's kernels through cs_recover_ex."""
    import numpy as np
    import paper_2604_14156_b200 as cs
    from gen import rng
    out = {}
    Phi = rng.normal(cfg.seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    mu = W.spectral_step(Phi)
    Pn = Phi.double()
    for k in sorted({max(1, cfg.k // 8), max(1, cfg.k // 4), max(1, cfg.k // 2), cfg.k}):
        plan = cs.Plan(cfg.d, cfg.d_ff, cfg.group, cfg.m, k, 40, torch.float32 if cfg.w_dtype == "f32" else torch.bfloat16,
                       trials, cfg.rms_eps)
        sup = rng.k_subset(cfg.seed, (97, k), cfg.G, k, rows=trials)
        c = rng.normal(cfg.seed, (98, k), (trials, k))
        c = torch.sign(c) * c.abs().clamp_min(0.5)
        y = torch.einsum("tk,tmk->tm", c, Pn[:, sup.long()].permute(1, 0, 2)).float().to(dev)
        row = {}
        for solver in ("iht", "niht", "omp"):
            if solver == "omp" and k > 64:
                continue
            got, _, _ = cs.cs_recover_ex(plan, Phi.to(dev), mu, y, cs.StepOptions(plan, trials, solver=solver, device=dev))
            row[solver] = float((got.cpu() == sup).all(dim=1).float().mean())
        out[f"k={k}"] = row
        plan.close()
    return {"m": cfg.m, "G": cfg.G, "trials": trials, "iterations": 40, "rate_by_sparsity": out}


def cpu_baseline(cfg, cpu_layers, hx, seconds: float, single: bool):
    """The fp64 oracle as it stands, on the host cores, on a bounded sample of the same steps: with
    all cores, and (for the headline workload) with one thread."""
    import oracle

    def sample(budget):
        n = 0
        t0 = time.perf_counter()
        while True:
            L = cpu_layers[n % len(cpu_layers)]
            oracle.layer_step(L, hx[n % hx.shape[0]], group=cfg.group, k=cfg.k, T=cfg.T, rms_eps=cfg.rms_eps)
            n += 1
            dt = time.perf_counter() - t0
            if dt >= budget or n >= 4096:
                return n, dt

    cores = oracle.num_threads()
    n, dt = sample(seconds)
    res = {"value": cfg.B * n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"{n} full steps (batch {cfg.B}) of the same workload over {len(cpu_layers)} layers, {dt:.1f} s"}
    if single:
        oracle.set_num_threads(1)
        try:
            n1, dt1 = sample(seconds)
        finally:
            oracle.set_num_threads(cores)
        res["single_thread"] = {"value": cfg.B * n1 / dt1, "unit": UNIT, "cores": 1,
                                "sample": f"{n1} full steps, {dt1:.1f} s"}
    return res


def cpu_baseline_prompt(cfg, L, H, seconds: float):
    """Oracle on the prompt workload: the support from the whole prompt's mean sketch, then the FFN of
    a 32-token subset over it (a full prompt takes the oracle several seconds)."""
    import oracle
    t0 = time.perf_counter()
    _, r = oracle.prompt_support(L.S, L.Phi, H.double().numpy(), cfg.k, cfg.T, L.mu)
    t_sup = time.perf_counter() - t0
    n = 0
    t0 = time.perf_counter()
    while True:
        oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, H[n % cfg.B].double().numpy(), r.support)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or n >= cfg.B:
            break
    per_prompt = t_sup + dt / n * cfg.B
    return {"value": cfg.B / per_prompt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"prompt support from all {cfg.B} tokens ({t_sup:.2f} s) + FFN of {n} tokens ({dt:.1f} s) scaled to {cfg.B}"}


def resolve(name: str, args=None):
    """'workload' or 'workload:k' -> Config (with the command line's overrides for the primary)."""
    base, _, k = name.partition(":")
    cfg = W.CONFIGS[base]
    if k:
        cfg = cfg.with_(k=int(k))
    if args is not None:
        if args.k:
            cfg = cfg.with_(k=args.k)
        if args.batch:
            cfg = cfg.with_(B=args.batch)
    return cfg


def run_ours(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    K, Wm = max(args.steps, 1), max(args.warmup, 3)
    cfg = resolve(args.workload, args)
    fn = bench_prompt if cfg.prompt else bench_decode
    out = fn(cfg, args, K, Wm, rank, world, local, dev, primary=True)
    # the other workloads, briefly, in the same run (one GPU: they say nothing new about scaling)
    if not args.no_extra and world == 1 and not (args.k or args.batch or args.crossover):
        extras = {}
        sub = argparse.Namespace(**vars(args))
        sub.layers = 0
        for name in EXTRA_WORKLOADS:
            c = resolve(name)
            if c.name == cfg.name and c.k == cfg.k:
                continue
            torch.cuda.empty_cache()
            k_extra = 20 if not c.prompt else 8
            f = bench_prompt if c.prompt else bench_decode
            r = f(c, sub, k_extra, 3, rank, world, local, dev, primary=False)
            for drop in ("metric", "unit", "n_gpus", "higher_is_better", "scaling", "vs_baseline", "data"):
                r.pop(drop, None)
            extras[name] = r
        out["workloads"] = extras
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_reference(args):
    """The CPU oracle as the reference arm: K steps on the host cores.  When K full steps would
    take more than a few minutes, each step runs the full sketch and recovery but the FFN over only
    the first kk of the k recovered groups, and the FFN time is scaled by k/kk."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    cfg = W.CONFIGS[args.workload]
    K, Wm = args.steps, max(args.warmup, 1)
    layers = [W.make_layer(cfg, i) for i in range(2)]
    xs = [W.make_tokens(cfg, layers[0].A, batch=j).h for j in range(4)]

    def pieces(i, kk):
        L = layers[i % 2]
        x = xs[i % 4].double().numpy()
        t0 = time.perf_counter()
        n = np.stack([oracle.rmsnorm(x[t], L.gamma, cfg.rms_eps) for t in range(cfg.B)]) if cfg.rms else x
        y = oracle.sketch(L.S, n)
        sups = [oracle.iht(L.Phi, y[t], cfg.k, cfg.T, L.mu).support for t in range(cfg.B)]
        t1 = time.perf_counter()
        for t in range(cfg.B):
            oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, n[t], sups[t][:kk])
        t2 = time.perf_counter()
        return t1 - t0, t2 - t1

    a, b = pieces(0, cfg.k)
    est = a + b
    budget = 150.0
    kk = cfg.k if est * (K + Wm) <= budget else max(1, int(cfg.k * budget / (est * (K + Wm))))
    for i in range(min(Wm, 3) if kk < cfg.k else Wm):
        pieces(i, kk)
    t_sr = t_ffn = 0.0
    for i in range(K):
        a, b = pieces(i, kk)
        t_sr += a; t_ffn += b
    total = t_sr + t_ffn * (cfg.k / kk)
    value = cfg.B * K / total
    sample = (f"{K} full steps" if kk == cfg.k else
              f"{K} steps, FFN over {kk} of {cfg.k} recovered groups per token, FFN time scaled by {cfg.k}/{kk}")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
        "warmup": Wm, "ms_per_step": total / K * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "d": cfg.d, "d_ff": cfg.d_ff, "groups": cfg.G, "group": cfg.group,
                   "m": cfg.m, "k": cfg.k, "T": cfg.T, "batch": cfg.B, "weights": cfg.w_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
