"""cs_ffn_exec_static: the gather FFN for callers that are not allowed to allocate device memory
(a host framework that owns the device heap, a fixed start-up memory budget, a section where the
implicit synchronisation of cudaMalloc is unacceptable).  It keeps its scratch in a fixed array
inside the library instead of a plan.  Checked here against cs_ffn_exec, the plan-based entry
point, on two calls in a row (the second call reuses the array with the first call's contents
still in it).  Collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import pytest
import torch

import paper_2604_14156_b200 as cs
from gen import rng, workloads as W
from parity_util import device_layer, make_plan, rel

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
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup, residual=res, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # both paths accumulate in f32 over the same rows; only the split over CTAs may differ
        assert rel(out.cpu().numpy(), want.cpu().numpy()) <= 1e-5
        nores = cs.cs_ffn_exec_static(cfg.d, cfg.d_ff, cfg.group, cfg.k, lay, h, sup)
        assert rel(nores.cpu().numpy(), (want - res).cpu().numpy()) <= 1e-4


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
