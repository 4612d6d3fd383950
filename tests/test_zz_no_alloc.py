"""cs_ffn_exec_static: the gather FFN for callers that are not allowed to allocate device memory
(a host framework that owns the device heap, a fixed start-up memory budget, a section where the
implicit synchronisation of cudaMalloc is unacceptable).  It keeps its scratch in a fixed array
inside the library instead of a plan.  Checked here against cs_ffn_exec, the plan-based entry
point, and against the CPU oracle, on two calls in a row (the second call reuses the array with the
first call's contents still in it).  Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import pytest
import torch

import oracle
import paper_2604_14156_b200 as cs
from gen import rng, workloads as W
from parity_util import TIGHT_TOL, device_layer, make_plan, rel

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("name,B", [("l2_7b_b1", 1), ("tiny_f32", 4)])
def test_static_scratch_entry_matches_plan_entry_twice(name, B):
    cfg = W.CONFIGS[name]
    L = W.make_layer(cfg, device=DEV)
    plan = make_plan(cfg, max_tokens=B)
    lay = device_layer(plan, L)
    for call in range(2):
        tk = W.make_tokens(cfg, L.A, batch=call, B=B)
        h, sup = tk.h.to(DEV), tk.planted.to(DEV)
        res = rng.normal(cfg.seed, (90 + call,), (B, cfg.d), dtype=torch.float32).to(DEV)
        want = cs.cs_ffn_exec(plan, lay, h, sup, residual=res)
        out = torch.empty_like(want)
        nores = torch.empty_like(want)
        if call == 0:   # the first call per device looks the array up (and may load the library's device code)
            cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup, residual=res, out=out)
        torch.cuda.synchronize()
        # the driver's own count of free device memory sees any allocation, the library's included
        free_before, _ = torch.cuda.mem_get_info()
        cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup, residual=res, out=out)
        cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup, out=nores)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        # both paths accumulate in f32 over the same rows; only the split over CTAs may differ
        assert rel(out.cpu().numpy(), want.cpu().numpy()) <= 1e-5
        assert rel(nores.cpu().numpy(), (want - res).cpu().numpy()) <= 1e-4
        Lc = L.to("cpu")
        for t in range(B):
            ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t], tk.planted[t])
            assert rel(nores[t].cpu().numpy(), ref) <= TIGHT_TOL[cfg.w_dtype]
            assert rel(out[t].cpu().numpy(), ref + res[t].cpu().double().numpy()) <= TIGHT_TOL[cfg.w_dtype]


def test_static_scratch_entry_checks_pointers_and_supports_on_the_way_in():
    """A pointer off the 16-byte grid is refused before anything runs (as cs_ffn_exec does); a group
    index outside [0, G) is never read through (its channels contribute zero)."""
    cfg = W.CONFIGS["tiny_f32"]
    L = W.make_layer(cfg, device=DEV)
    plan = make_plan(cfg, max_tokens=2)
    lay = device_layer(plan, L)
    tk = W.make_tokens(cfg, L.A, B=2)
    h, sup = tk.h.to(DEV), tk.planted.to(DEV)
    shifted = torch.zeros(2 * cfg.d + 4, device=DEV)[1:1 + 2 * cfg.d].view(2, cfg.d)   # 4-byte offset
    shifted.copy_(h)
    for kw in (dict(h=shifted), dict(out=shifted), dict(residual=shifted)):
        args = dict(h=h, out=torch.empty_like(h), residual=None)
        args.update(kw)
        with pytest.raises(cs.CSError) as e:
            cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, args["h"], sup, residual=args["residual"],
                                  out=args["out"])
        assert e.value.code == 3
    bad = sup.clone()
    bad[1, 0] = -1
    bad[1, cfg.k - 1] = cfg.G
    out = cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, bad).cpu().numpy()
    Lc = L.to("cpu")
    ref0 = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[0], tk.planted[0])
    ref1 = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[1], tk.planted[1][1:cfg.k - 1])
    assert rel(out[0], ref0) <= TIGHT_TOL["f32"] and rel(out[1], ref1) <= TIGHT_TOL["f32"]


def test_static_scratch_entry_rejects_oversized_batches():
    cfg = W.CONFIGS["l2_7b_b1"]
    L = W.make_layer(cfg, device=DEV)
    plan = make_plan(cfg, max_tokens=1)
    lay = device_layer(plan, L)
    B = 6  # 6 tokens x 88 CTAs x 4096 floats exceed the 8 MiB array
    h = torch.zeros(B, cfg.d, device=DEV)
    sup = torch.arange(cfg.k, dtype=torch.int32, device=DEV).repeat(B, 1)
    with pytest.raises(cs.CSError) as e:
        cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup)
    assert e.value.code == 2
