"""The C boundary without a GPU: the library loads, exports what include/cs.h declares, and
rejects bad configurations on the host before touching CUDA."""
import ctypes
import os

import pytest
import torch

import paper_2604_14156_b200 as cs
from paper_2604_14156_b200 import binding, build


@pytest.fixture(scope="module")
def lib():
    build.build()
    return cs.load_library()


def test_library_exports_every_declared_symbol(lib):
    names = cs.exported_symbols()
    assert {"cs_plan_create", "cs_plan_destroy", "cs_sketch", "cs_recover", "cs_ffn_exec", "cs_layer_step",
            "cs_prompt_support", "cs_ffn_exec_shared", "cs_last_device_status", "cs_status_string",
            "cs_recover_warm"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    seen = {lib.cs_status_string(i) for i in range(8)}
    assert len(seen) == 8 and b"ok" in seen


@pytest.mark.parametrize("kw,code", [
    (dict(d=0), 2), (dict(d_ff=1000), 2), (dict(k=0), 2), (dict(k=17), 2), (dict(T=-1), 2),
    (dict(max_tokens=0), 2), (dict(group=32, d_ff=1024), 3), (dict(d=200), 3), (dict(m=65), 3),
    (dict(d_ff=64 * 129), 3), (dict(d=16384), 3), (dict(w_dtype=torch.float16), 3),
    (dict(rms_eps=0.0), 5), (dict(rms_eps=float("nan")), 5),
])
def test_plan_create_rejects_bad_configs_on_the_host(lib, kw, code):
    args = dict(d=256, d_ff=1024, group=64, m=8, k=4, T=10, w_dtype=torch.float32, max_tokens=4, rms_eps=1e-5)
    args.update(kw)
    with pytest.raises(cs.CSError) as e:
        cs.Plan(**args)
    assert e.value.code == code


def test_null_arguments_are_reported(lib):
    assert lib.cs_plan_create(None, None) == 1
    assert lib.cs_plan_destroy(None) == 1
    assert lib.cs_sketch(None, None, None, 1, None, None) == 1
    assert lib.cs_recover(None, None, 1.0, None, 1, None, None, None, None) == 1
    assert lib.cs_recover_warm(None, None, 1.0, None, 1, 1, None, None, None, None, None, None) == 1
    assert lib.cs_uds_budget(None, None, 1, 8, 1.0, 1.0, 1, 2, None, None, None) == 1
    assert lib.cs_support_drift(None, None, None, 1, None, None) == 1
    assert lib.cs_layer_step(None, None, None, 1, None, None, None, None, None) == 1
    assert lib.cs_launch_count(None) == 0


def test_binding_refuses_cpu_tensors():
    with pytest.raises(TypeError):
        binding._ptr(torch.zeros(4), torch.float32, "x")


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.load_library()
