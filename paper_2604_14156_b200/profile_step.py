"""Runs a handful of steps of one workload and exits: the command to put under a profiler.

    python -m paper_2604_14156_b200.profile_step --workload l2_7b_b1 --steps 8 [--layers 3] [--batch B] [--k K]
                                                 [--entry step|exec] [--speculative]

Unlike bench.py there is no timing loop, no CUDA graph and no CPU baseline: `--warmup` untimed steps,
then `--steps` steps launched one after the other over `--layers` distinct layers (a few hundred MB
on the device, more than the L2 holds, so DRAM counters still mean something), one synchronisation,
done.  `--entry exec` calls the actuator alone (cs_ffn_exec, or cs_ffn_exec_shared for the prompt
workload) on the supports of a finished step.
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import paper_2604_14156_b200 as cs  # noqa: E402
from gen import workloads as W  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="l2_7b_b1", choices=sorted(W.CONFIGS))
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--layers", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--entry", choices=["step", "exec"], default="step")
    ap.add_argument("--speculative", action="store_true")
    a = ap.parse_args()
    cfg = W.CONFIGS[a.workload]
    if a.k:
        cfg = cfg.with_(k=a.k)
    if a.batch:
        cfg = cfg.with_(B=a.batch)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    plan = cs.Plan(cfg.d, cfg.d_ff, cfg.group, cfg.m, cfg.k, cfg.T,
                   torch.float32 if cfg.w_dtype == "f32" else torch.bfloat16, cfg.B, cfg.rms_eps)
    if a.speculative:
        plan.set_speculative(True)
    raw = [W.make_layer(cfg, i, device=dev) for i in range(a.layers)]
    layers = [cs.Layer(plan, L.S, L.Phi, L.W_gate, L.W_up, L.Wd_t, L.mu, L.gamma, cfg.rms) for L in raw]
    xs = [W.make_tokens(cfg, raw[0].A, batch=j).h.to(dev) for j in range(4)]
    if cfg.prompt:
        out = torch.empty_like(xs[0])
        sup, _, _ = cs.cs_prompt_support(plan, raw[0].S, raw[0].Phi, raw[0].mu, xs[0])

        def step(i):
            L = raw[i % a.layers]
            if a.entry == "step":
                s, _, _ = cs.cs_prompt_support(plan, L.S, L.Phi, L.mu, xs[i % 4])
            else:
                s = sup
            cs.cs_ffn_exec_shared(plan, layers[i % a.layers], xs[i % 4], s, out=out)
    else:
        out = torch.empty_like(xs[0])
        _, sup, _, _ = cs.cs_layer_step(plan, layers[0], xs[0])

        def step(i):
            if a.entry == "step":
                cs.cs_layer_step(plan, layers[i % a.layers], xs[i % 4], x_out=out, want_aux=False)
            else:
                cs.cs_ffn_exec(plan, layers[i % a.layers], xs[i % 4], sup, out=out)
    for i in range(a.warmup + a.steps):
        step(i)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    print(f"{a.workload}: {a.steps} steps after {a.warmup}, {plan.launches} launches in all")


if __name__ == "__main__":
    main()
