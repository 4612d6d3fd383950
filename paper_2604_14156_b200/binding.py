"""ctypes binding of libcs_b200.so (argument marshalling only)."""
from __future__ import annotations

import ctypes
import os
import re
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libcs_b200.so")
_HEADER = os.path.join(os.path.dirname(_PKG), "include", "cs.h")

CS_F32, CS_BF16 = 0, 1
_STATUS_NAMES = {0: "CS_OK", 1: "CS_ERR_NULL", 2: "CS_ERR_SHAPE", 3: "CS_ERR_UNSUPPORTED",
                 4: "CS_ERR_SUPPORT", 5: "CS_ERR_NONFINITE", 6: "CS_ERR_CUDA", 7: "CS_ERR_TIMEOUT"}


class CSError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {_STATUS_NAMES.get(code, code)}" + (f" ({detail})" if detail else ""))


class _Config(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("group", ctypes.c_int32),
                ("m", ctypes.c_int32), ("k", ctypes.c_int32), ("T", ctypes.c_int32),
                ("w_dtype", ctypes.c_int32), ("max_tokens", ctypes.c_int32), ("rms_eps", ctypes.c_float)]


class _StepOptions(ctypes.Structure):
    _fields_ = [("solver", ctypes.c_int32), ("T", ctypes.c_int32), ("support_prev", ctypes.c_void_p),
                ("z_prev", ctypes.c_void_p), ("warm_start", ctypes.c_int32), ("gamma", ctypes.c_float),
                ("reuse_support", ctypes.c_int32), ("srht_sign", ctypes.c_void_p), ("srht_rows", ctypes.c_void_p),
                ("delta_out", ctypes.c_void_p), ("drift_out", ctypes.c_void_p)]


SOLVERS = {"iht": 0, "niht": 1, "omp": 2}


class _Layer(ctypes.Structure):
    _fields_ = [("S", ctypes.c_void_p), ("Phi", ctypes.c_void_p), ("W_gate", ctypes.c_void_p),
                ("W_up", ctypes.c_void_p), ("Wd_t", ctypes.c_void_p), ("rms_gamma", ctypes.c_void_p),
                ("mu", ctypes.c_float), ("add_residual", ctypes.c_int32)]


def library_path() -> str:
    return _LIB_PATH


def exported_symbols():
    """Names of the functions include/cs.h declares (used by the load test)."""
    text = open(_HEADER).read()
    return sorted(set(re.findall(r"\b(cs_[a-z_]+)\s*\(", text)))


_lib = None


def load_library():
    """Load libcs_b200.so; there is no fallback if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2604_14156_b200.build` "
                          "(there is no CPU path)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
    lib.cs_plan_create.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp)]
    lib.cs_plan_destroy.argtypes = [vp]
    lib.cs_sketch.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.cs_recover.argtypes = [vp, vp, f32, vp, i32, vp, vp, vp, vp]
    lib.cs_recover_warm.argtypes = [vp, vp, f32, vp, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.cs_uds_budget.argtypes = [vp, vp, i32, i32, f32, f32, i32, i32, vp, vp, vp]
    lib.cs_support_drift.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.cs_ffn_exec.argtypes = [vp, ctypes.POINTER(_Layer), vp, vp, i32, vp, vp, vp]
    lib.cs_layer_step.argtypes = [vp, ctypes.POINTER(_Layer), vp, i32, vp, vp, vp, vp, vp]
    lib.cs_prompt_support.argtypes = [vp, vp, vp, f32, vp, i32, vp, vp, vp, vp]
    lib.cs_ffn_exec_shared.argtypes = [vp, ctypes.POINTER(_Layer), vp, i32, vp, vp, vp]
    lib.cs_layer_step_host.argtypes = [vp, ctypes.POINTER(_Layer), vp, i32, vp, vp, vp]
    lib.cs_plan_enable_timing.argtypes = [vp, i32]
    lib.cs_plan_set_crossover.argtypes = [vp, i32]
    lib.cs_plan_set_crossover.restype = ctypes.c_int
    lib.cs_plan_set_speculative.argtypes = [vp, i32]
    lib.cs_plan_set_speculative.restype = ctypes.c_int
    lib.cs_plan_crossover.argtypes = [vp]
    lib.cs_plan_crossover.restype = ctypes.c_int32
    lib.cs_plan_stage_times.argtypes = [vp, vp, ctypes.POINTER(f32 * 5)]
    lib.cs_support_drift_ratio.argtypes = [vp, vp, vp, i32, vp, vp, vp]
    lib.cs_recover_ex.argtypes = [vp, vp, f32, vp, i32, ctypes.POINTER(_StepOptions), vp, vp, vp, vp]
    lib.cs_sketch_srht.argtypes = [vp, vp, vp, vp, i32, vp, vp]
    lib.cs_layer_step_ex.argtypes = [vp, ctypes.POINTER(_Layer), vp, i32, ctypes.POINTER(_StepOptions), vp, vp, vp, vp, vp]
    lib.cs_layer_step_fallback.argtypes = [vp, vp, ctypes.POINTER(_Layer), vp, i32, ctypes.POINTER(_StepOptions), f32, vp,
                                           vp, vp, vp, vp, ctypes.POINTER(i32), vp]
    for name in ("cs_support_drift_ratio", "cs_recover_ex", "cs_sketch_srht", "cs_layer_step_ex", "cs_layer_step_fallback"):
        getattr(lib, name).restype = ctypes.c_int
    lib.cs_ffn_exec_static.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(_Layer), vp, vp, i32, vp, vp, vp]
    lib.cs_ffn_exec_static.restype = ctypes.c_int
    lib.cs_bucket.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.cs_bucket.restype = ctypes.c_int
    lib.cs_last_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.cs_launch_count.argtypes = [vp]
    lib.cs_launch_count.restype = ctypes.c_int64
    lib.cs_last_cuda_error.argtypes = [vp]
    lib.cs_last_cuda_error.restype = ctypes.c_char_p
    lib.cs_status_string.argtypes = [ctypes.c_int]
    lib.cs_status_string.restype = ctypes.c_char_p
    for name in ("cs_plan_create", "cs_plan_destroy", "cs_sketch", "cs_recover", "cs_ffn_exec",
                 "cs_layer_step", "cs_prompt_support", "cs_ffn_exec_shared", "cs_last_device_status",
                 "cs_layer_step_host", "cs_plan_enable_timing", "cs_plan_stage_times", "cs_recover_warm", "cs_uds_budget",
                 "cs_support_drift"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str, shape=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


class Plan:
    """Owns a cs_plan (device scratch sized for one layer shape)."""

    def __init__(self, d: int, d_ff: int, group: int, m: int, k: int, T: int, w_dtype: torch.dtype,
                 max_tokens: int, rms_eps: float = 1e-5):
        self.lib = load_library()
        self.d, self.d_ff, self.group, self.m, self.k, self.T = d, d_ff, group, m, k, T
        self.G = d_ff // group if group > 0 else 0
        self.w_dtype = w_dtype
        self.max_tokens = max_tokens
        code = {torch.float32: CS_F32, torch.bfloat16: CS_BF16}.get(w_dtype, -1)
        cfg = _Config(d, d_ff, group, m, k, T, code, max_tokens, rms_eps)
        handle = ctypes.c_void_p()
        st = self.lib.cs_plan_create(ctypes.byref(cfg), ctypes.byref(handle))
        self.handle = None
        if st != 0:
            raise CSError(st, "cs_plan_create")
        self.handle = handle

    def check(self, st: int, where: str):
        if st != 0:
            detail = self.lib.cs_last_cuda_error(self.handle).decode() if st == 6 else ""
            raise CSError(st, where, detail)

    def device_status(self, stream=None) -> int:
        code = ctypes.c_int32(0)
        self.check(self.lib.cs_last_device_status(self.handle, _stream(stream), ctypes.byref(code)),
                   "cs_last_device_status")
        return code.value

    @property
    def crossover(self) -> int:
        """Smallest decode batch that runs on the tensor cores."""
        return int(self.lib.cs_plan_crossover(self.handle))

    def set_crossover(self, tokens: int):
        self.check(self.lib.cs_plan_set_crossover(self.handle, int(tokens)), "cs_plan_set_crossover")

    def set_speculative(self, on=True):
        """Small batches, on the recovery's first iterate: 1 / True = start the gather FFN's weight stream,
        2 = only warm L2 with its weight blocks, 0 = the plain chain (see include/cs.h)."""
        self.check(self.lib.cs_plan_set_speculative(self.handle, int(on)), "cs_plan_set_speculative")

    def enable_timing(self, on: bool = True):
        self.check(self.lib.cs_plan_enable_timing(self.handle, int(on)), "cs_plan_enable_timing")

    def stage_times(self, stream=None):
        """Milliseconds of (sketch, recover, exec, reduce, exec2) in the most recent call; exec2 is
        the down GEMM of the tensor-core decode path (0 otherwise)."""
        ms = (ctypes.c_float * 5)()
        self.check(self.lib.cs_plan_stage_times(self.handle, _stream(stream), ctypes.byref(ms)),
                   "cs_plan_stage_times")
        return tuple(ms)

    @property
    def launches(self) -> int:
        return int(self.lib.cs_launch_count(self.handle))

    def close(self):
        if self.handle is not None:
            self.lib.cs_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Layer:
    """Device tensors of one layer; keeps them alive and exposes the C struct."""

    def __init__(self, plan: Plan, S, Phi, W_gate, W_up, Wd_t, mu: float, rms_gamma=None,
                 add_residual: bool = False):
        G = plan.G
        self.tensors = (S, Phi, W_gate, W_up, Wd_t, rms_gamma)
        self.c = _Layer(
            _ptr(S, torch.float32, "S", (plan.m, plan.d)), _ptr(Phi, torch.float32, "Phi", (plan.m, G)),
            _ptr(W_gate, plan.w_dtype, "W_gate", (plan.d_ff, plan.d)),
            _ptr(W_up, plan.w_dtype, "W_up", (plan.d_ff, plan.d)),
            _ptr(Wd_t, plan.w_dtype, "Wd_t", (plan.d_ff, plan.d)),
            _ptr(rms_gamma, torch.float32, "rms_gamma", (plan.d,)), float(mu), int(bool(add_residual)))
        self.mu = float(mu)
        self.S, self.Phi = S, Phi


def cs_sketch(plan: Plan, S, h, y=None, stream=None):
    B = h.shape[0]
    y = torch.empty((B, plan.m), dtype=torch.float32, device=h.device) if y is None else y
    plan.check(plan.lib.cs_sketch(plan.handle, _ptr(S, torch.float32, "S", (plan.m, plan.d)),
                                  _ptr(h, torch.float32, "h", (B, plan.d)), B,
                                  _ptr(y, torch.float32, "y", (B, plan.m)), _stream(stream)), "cs_sketch")
    return y


def cs_recover(plan: Plan, Phi, mu: float, y, stream=None):
    B = y.shape[0]
    dev = y.device
    support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
    z = torch.empty((B, plan.k), dtype=torch.float32, device=dev)
    resid = torch.empty((B,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_recover(plan.handle, _ptr(Phi, torch.float32, "Phi", (plan.m, plan.G)), float(mu),
                                   _ptr(y, torch.float32, "y", (B, plan.m)), B, support.data_ptr(),
                                   z.data_ptr(), resid.data_ptr(), _stream(stream)), "cs_recover")
    return support, z, resid


def cs_recover_warm(plan: Plan, Phi, mu: float, y, T: int, support0, z0, stream=None):
    """T iterations from the k-sparse iterate (support0, z0) instead of zero; returns (support, z, resid)."""
    B = y.shape[0]
    dev = y.device
    support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
    z = torch.empty((B, plan.k), dtype=torch.float32, device=dev)
    resid = torch.empty((B,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_recover_warm(plan.handle, _ptr(Phi, torch.float32, "Phi", (plan.m, plan.G)), float(mu),
                                        _ptr(y, torch.float32, "y", (B, plan.m)), B, int(T),
                                        _ptr(support0, torch.int32, "support0", (B, plan.k)),
                                        _ptr(z0, torch.float32, "z0", (B, plan.k)), support.data_ptr(),
                                        z.data_ptr(), resid.data_ptr(), _stream(stream)), "cs_recover_warm")
    return support, z, resid


def cs_support_drift(plan: Plan, support_prev, support_cur, stream=None):
    """|S_t symmetric-difference S_{t-1}| per token for two [B, k] int32 support lists."""
    B = support_cur.shape[0]
    drift = torch.empty((B,), dtype=torch.int32, device=support_cur.device)
    plan.check(plan.lib.cs_support_drift(plan.handle, _ptr(support_prev, torch.int32, "support_prev", (B, plan.k)),
                                         _ptr(support_cur, torch.int32, "support_cur", (B, plan.k)), B,
                                         drift.data_ptr(), _stream(stream)), "cs_support_drift")
    return drift


def cs_support_drift_ratio(plan: Plan, support_prev, support_cur, stream=None):
    """(Delta_t [B] int32, D_t [B] float32): the drift count and the normalised drift of Sec. 15."""
    B = support_cur.shape[0]
    delta = torch.empty((B,), dtype=torch.int32, device=support_cur.device)
    D = torch.empty((B,), dtype=torch.float32, device=support_cur.device)
    plan.check(plan.lib.cs_support_drift_ratio(plan.handle, _ptr(support_prev, torch.int32, "support_prev", (B, plan.k)),
                                               _ptr(support_cur, torch.int32, "support_cur", (B, plan.k)), B,
                                               delta.data_ptr(), D.data_ptr(), _stream(stream)), "cs_support_drift_ratio")
    return delta, D


class StepOptions:
    """Options of cs_recover_ex / cs_layer_step_ex; keeps the tensors it points at alive."""

    def __init__(self, plan: Plan, B: int, solver: str = "iht", T: int = -1, support_prev=None, z_prev=None,
                 warm_start: bool = False, gamma: float = 0.0, reuse_support: bool = False, srht=None,
                 want_drift: bool = False, device="cuda"):
        self.delta = self.drift = None
        if want_drift:
            self.delta = torch.empty((B,), dtype=torch.int32, device=device)
            self.drift = torch.empty((B,), dtype=torch.float32, device=device)
        self.keep = (support_prev, z_prev, srht)
        sign, rows = (None, None) if srht is None else srht
        self.c = _StepOptions(
            SOLVERS[solver], int(T), _ptr(support_prev, torch.int32, "support_prev", (B, plan.k)),
            _ptr(z_prev, torch.float32, "z_prev", (B, plan.k)), int(bool(warm_start)), float(gamma),
            int(bool(reuse_support)), _ptr(sign, torch.int32, "srht sign bits", (plan.d // 32,)),
            _ptr(rows, torch.int32, "srht rows", (plan.m,)),
            None if self.delta is None else self.delta.data_ptr(), None if self.drift is None else self.drift.data_ptr())


def cs_recover_ex(plan: Plan, Phi, mu: float, y, options: StepOptions, stream=None):
    B = y.shape[0]
    dev = y.device
    support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
    z = torch.empty((B, plan.k), dtype=torch.float32, device=dev)
    resid = torch.empty((B,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_recover_ex(plan.handle, _ptr(Phi, torch.float32, "Phi", (plan.m, plan.G)), float(mu),
                                      _ptr(y, torch.float32, "y", (B, plan.m)), B, ctypes.byref(options.c),
                                      support.data_ptr(), z.data_ptr(), resid.data_ptr(), _stream(stream)), "cs_recover_ex")
    return support, z, resid


def cs_sketch_srht(plan: Plan, sign_bits, rows, h, stream=None):
    """y [B, m] of the subsampled randomized Hadamard sketch; sign_bits [d/32] int32 (bit i set: s_i = -1), rows [m] int32."""
    B = h.shape[0]
    y = torch.empty((B, plan.m), dtype=torch.float32, device=h.device)
    plan.check(plan.lib.cs_sketch_srht(plan.handle, _ptr(sign_bits, torch.int32, "sign_bits", (plan.d // 32,)),
                                       _ptr(rows, torch.int32, "rows", (plan.m,)), _ptr(h, torch.float32, "h", (B, plan.d)),
                                       B, y.data_ptr(), _stream(stream)), "cs_sketch_srht")
    return y


def cs_layer_step_ex(plan: Plan, layer: Layer, x, options: StepOptions, x_out=None, stream=None):
    """Returns (x_out, support, z, resid)."""
    B = x.shape[0]
    dev = x.device
    x_out = torch.empty_like(x) if x_out is None else x_out
    support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
    z = torch.zeros((B, plan.k), dtype=torch.float32, device=dev)
    resid = torch.zeros((B,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_layer_step_ex(plan.handle, ctypes.byref(layer.c), _ptr(x, torch.float32, "x", (B, plan.d)), B,
                                         ctypes.byref(options.c), _ptr(x_out, torch.float32, "x_out", (B, plan.d)),
                                         support.data_ptr(), z.data_ptr(), resid.data_ptr(), _stream(stream)),
               "cs_layer_step_ex")
    return x_out, support, z, resid


def cs_layer_step_fallback(plan: Plan, dense: Plan, layer: Layer, x, tau: float, options: Optional[StepOptions] = None,
                           stream=None):
    """Returns (x_out, support, z, resid, flags, n_fallback); synchronises the stream (see include/cs.h)."""
    B = x.shape[0]
    dev = x.device
    x_out = torch.empty_like(x)
    support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
    z = torch.empty((B, plan.k), dtype=torch.float32, device=dev)
    resid = torch.empty((B,), dtype=torch.float32, device=dev)
    flags = torch.empty((B,), dtype=torch.int32, device=dev)
    n = ctypes.c_int32(0)
    plan.check(plan.lib.cs_layer_step_fallback(plan.handle, dense.handle, ctypes.byref(layer.c),
                                               _ptr(x, torch.float32, "x", (B, plan.d)), B,
                                               None if options is None else ctypes.byref(options.c), float(tau),
                                               x_out.data_ptr(), support.data_ptr(), z.data_ptr(), resid.data_ptr(),
                                               flags.data_ptr(), ctypes.byref(n), _stream(stream)), "cs_layer_step_fallback")
    return x_out, support, z, resid, flags, n.value


def cs_uds_budget(plan: Plan, logits, m_base: float, gamma: float, m_min: int, m_max: int, stream=None):
    """Entropy of softmax(logits[t]) and the budget clip(floor(m_base (1 + gamma H)), m_min, m_max); returns (m_t, H)."""
    B, V = logits.shape
    H = torch.empty((B,), dtype=torch.float32, device=logits.device)
    m_t = torch.empty((B,), dtype=torch.int32, device=logits.device)
    plan.check(plan.lib.cs_uds_budget(plan.handle, _ptr(logits, torch.float32, "logits", (B, V)), B, V, float(m_base),
                                      float(gamma), int(m_min), int(m_max), H.data_ptr(), m_t.data_ptr(),
                                      _stream(stream)), "cs_uds_budget")
    return m_t, H


def cs_ffn_exec(plan: Plan, layer: Layer, h, support, residual=None, out=None, stream=None):
    B = h.shape[0]
    out = torch.empty((B, plan.d), dtype=torch.float32, device=h.device) if out is None else out
    plan.check(plan.lib.cs_ffn_exec(plan.handle, ctypes.byref(layer.c), _ptr(h, torch.float32, "h", (B, plan.d)),
                                    _ptr(support, torch.int32, "support", (B, plan.k)), B,
                                    _ptr(residual, torch.float32, "residual", (B, plan.d)),
                                    _ptr(out, torch.float32, "out", (B, plan.d)), _stream(stream)), "cs_ffn_exec")
    return out


def cs_ffn_exec_static(d: int, d_ff: int, group: int, k: int, layer: Layer, h, support, residual=None, out=None,
                       stream=None):
    """The gather FFN without a plan and without any device allocation by the library.

    For callers that may not allocate on the device (see include/cs.h): the scratch is a fixed
    8 MiB array inside the library.  ``out`` must be passed by such callers; it is only created
    here, with torch, as a convenience for tests.  Raises CSError(CS_ERR_SHAPE) when B is too
    large for the fixed array.
    """
    lib = load_library()
    w_dtype = layer.tensors[2].dtype
    code = {torch.float32: CS_F32, torch.bfloat16: CS_BF16}.get(w_dtype, -1)
    cfg = _Config(d, d_ff, group, 1, k, 0, code, 1, 1e-5)
    B = h.shape[0]
    out = torch.empty((B, d), dtype=torch.float32, device=h.device) if out is None else out
    st = lib.cs_ffn_exec_static(ctypes.byref(cfg), ctypes.byref(layer.c), _ptr(h, torch.float32, "h", (B, d)),
                                _ptr(support, torch.int32, "support", (B, k)), B,
                                _ptr(residual, torch.float32, "residual", (B, d)),
                                _ptr(out, torch.float32, "out", (B, d)), _stream(stream))
    if st != 0:
        raise CSError(st, "cs_ffn_exec_static")
    return out


def cs_bucket(plan: Plan, support, stream=None):
    """(counts [G], offsets [G+1], token_ids [B*k]) of the group -> tokens inversion."""
    B = support.shape[0]
    dev = support.device
    counts = torch.empty((plan.G,), dtype=torch.int32, device=dev)
    offsets = torch.empty((plan.G + 1,), dtype=torch.int32, device=dev)
    token_ids = torch.empty((B * plan.k,), dtype=torch.int32, device=dev)
    plan.check(plan.lib.cs_bucket(plan.handle, _ptr(support, torch.int32, "support", (B, plan.k)), B,
                                  counts.data_ptr(), offsets.data_ptr(), token_ids.data_ptr(), _stream(stream)),
               "cs_bucket")
    return counts, offsets, token_ids


def cs_layer_step(plan: Plan, layer: Layer, x, x_out=None, want_aux: bool = True, stream=None):
    """Returns (x_out, support, z, resid); the last three are None when want_aux is False."""
    B = x.shape[0]
    dev = x.device
    x_out = torch.empty_like(x) if x_out is None else x_out
    support = z = resid = None
    if want_aux:
        support = torch.empty((B, plan.k), dtype=torch.int32, device=dev)
        z = torch.empty((B, plan.k), dtype=torch.float32, device=dev)
        resid = torch.empty((B,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_layer_step(plan.handle, ctypes.byref(layer.c), _ptr(x, torch.float32, "x", (B, plan.d)), B,
                                      _ptr(x_out, torch.float32, "x_out", (B, plan.d)),
                                      None if support is None else support.data_ptr(),
                                      None if z is None else z.data_ptr(),
                                      None if resid is None else resid.data_ptr(), _stream(stream)),
               "cs_layer_step")
    return x_out, support, z, resid


def cs_layer_step_host(plan: Plan, layer: Layer, x_host, x_out_host, support_host=None, stream=None):
    """x_host / x_out_host: CPU float32 tensors [B, d] (pinned for asynchronous copies)."""
    B = x_host.shape[0]
    for t, name in ((x_host, "x_host"), (x_out_host, "x_out_host")):
        if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != (B, plan.d):
            raise TypeError(f"{name} must be a contiguous CPU float32 tensor of shape ({B}, {plan.d})")
    plan.check(plan.lib.cs_layer_step_host(plan.handle, ctypes.byref(layer.c), x_host.data_ptr(), B,
                                           x_out_host.data_ptr(),
                                           None if support_host is None else support_host.data_ptr(),
                                           _stream(stream)), "cs_layer_step_host")
    return x_out_host


def cs_prompt_support(plan: Plan, S, Phi, mu: float, H, stream=None):
    n = H.shape[0]
    dev = H.device
    support = torch.empty((plan.k,), dtype=torch.int32, device=dev)
    z = torch.empty((plan.k,), dtype=torch.float32, device=dev)
    resid = torch.empty((1,), dtype=torch.float32, device=dev)
    plan.check(plan.lib.cs_prompt_support(plan.handle, _ptr(S, torch.float32, "S", (plan.m, plan.d)),
                                          _ptr(Phi, torch.float32, "Phi", (plan.m, plan.G)), float(mu),
                                          _ptr(H, torch.bfloat16, "H", (n, plan.d)), n, support.data_ptr(),
                                          z.data_ptr(), resid.data_ptr(), _stream(stream)), "cs_prompt_support")
    return support, z, resid


def cs_ffn_exec_shared(plan: Plan, layer: Layer, H, support, out=None, stream=None):
    n = H.shape[0]
    out = torch.empty_like(H) if out is None else out
    plan.check(plan.lib.cs_ffn_exec_shared(plan.handle, ctypes.byref(layer.c),
                                           _ptr(H, torch.bfloat16, "H", (n, plan.d)), n,
                                           _ptr(support, torch.int32, "support", (plan.k,)),
                                           _ptr(out, torch.bfloat16, "out", (n, plan.d)), _stream(stream)),
               "cs_ffn_exec_shared")
    return out
