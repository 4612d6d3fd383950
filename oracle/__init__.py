"""ctypes front end of the fp64 CPU oracle (``cs_oracle.c``) plus the brute-force support search.

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this package and
shares no code with it.

Arrays go in and out as numpy; torch tensors are accepted for parameters
(float32, or bfloat16 read bit-exactly as uint16).  See ``cs_oracle.c`` for the
passage of the paper each function follows.
"""
from __future__ import annotations

import ctypes
import itertools
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "cs_oracle.c")
_LIB = os.path.join(_DIR, "libcs_oracle.so")

F32, BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile cs_oracle.c with gcc (OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(ctypes.c_int(n))


# ----------------------------------------------------------------------------- marshalling
def _f64(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().to("cpu").double().numpy()
    return np.ascontiguousarray(a, dtype=np.float64)


def _f32(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().to("cpu").numpy()
    a = np.asarray(a)
    if a.dtype != np.float32:
        raise TypeError(f"expected float32 parameter, got {a.dtype}")
    return np.ascontiguousarray(a)


def _i32(a) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().to("cpu").numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _weights(w):
    """(numpy array that keeps the memory alive, dtype code) for an f32 / bf16 weight tensor."""
    if hasattr(w, "detach"):
        import torch
        w = w.detach().to("cpu").contiguous()
        if w.dtype == torch.bfloat16:
            return w.view(torch.int16).numpy().view(np.uint16), BF16
        if w.dtype == torch.float32:
            return w.numpy(), F32
        raise TypeError(f"unsupported weight dtype {w.dtype}")
    w = np.ascontiguousarray(w)
    if w.dtype == np.float32:
        return w, F32
    if w.dtype == np.uint16:
        return w, BF16
    raise TypeError(f"unsupported weight dtype {w.dtype}")


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


# ----------------------------------------------------------------------------- functions
def rmsnorm(x, gamma, eps: float) -> np.ndarray:
    x = _f64(x); g = _f32(gamma)
    out = np.empty_like(x)
    rows = x.reshape(-1, x.shape[-1]); o = out.reshape(rows.shape)
    for i in range(rows.shape[0]):
        xi = np.ascontiguousarray(rows[i]); oi = np.empty_like(xi)
        lib().oracle_rmsnorm(_p(xi), _p(g), ctypes.c_int(xi.shape[0]), ctypes.c_double(eps), _p(oi))
        o[i] = oi
    return out


def sketch(S, h) -> np.ndarray:
    """y = S h for one vector [d] or a batch [B, d]."""
    S = _f32(S); h = _f64(h)
    m, d = S.shape
    rows = h.reshape(-1, d)
    y = np.empty((rows.shape[0], m))
    for i in range(rows.shape[0]):
        yi = np.empty(m)
        lib().oracle_sketch(_p(S), _p(np.ascontiguousarray(rows[i])), ctypes.c_int(m), ctypes.c_int(d), _p(yi))
        y[i] = yi
    return y.reshape(h.shape[:-1] + (m,))


def hard_threshold(v, k: int):
    """(keep mask [G] bool, gap) of H_k under the order |v| descending, index ascending."""
    v = _f64(v); G = v.shape[0]
    keep = np.zeros(G, dtype=np.int32); gap = ctypes.c_double(0.0)
    lib().oracle_hard_threshold(_p(v), ctypes.c_int(G), ctypes.c_int(k), _p(keep), ctypes.byref(gap))
    return keep.astype(bool), gap.value


class IHTResult:
    __slots__ = ("z", "support", "resid_hist", "gap_hist")

    def __init__(self, z, support, resid_hist, gap_hist):
        self.z, self.support, self.resid_hist, self.gap_hist = z, support, resid_hist, gap_hist

    @property
    def min_gap(self) -> float:
        return float(self.gap_hist.min()) if self.gap_hist.size else float("inf")

    @property
    def resid(self) -> float:
        return float(self.resid_hist[-1])


def iht(Phi, y, k: int, T: int, mu: float, z0=None) -> IHTResult:
    Phi = _f32(Phi); y = _f64(y)
    m, G = Phi.shape
    z = np.empty(G); sup = np.empty(k, dtype=np.int32)
    rh = np.empty(T + 1); gh = np.empty(max(T, 1))
    z0a = None if z0 is None else _f64(z0)
    lib().oracle_iht(_p(Phi), _p(y), ctypes.c_int(m), ctypes.c_int(G), ctypes.c_int(k), ctypes.c_int(T),
                     ctypes.c_double(mu), _p(z0a), _p(z), _p(sup), _p(rh), _p(gh))
    return IHTResult(z, sup, rh, gh[:T])


def iht_temporal(Phi, y, k: int, T: int, mu: float, gamma: float, z_prev, z0=None) -> IHTResult:
    """IHT on 1/2 ||y - Phi z||^2 + gamma ||z - z_prev||^2 (Sec. 5 temporal regulariser); z_prev, z0 dense [G]."""
    Phi = _f32(Phi); y = _f64(y)
    m, G = Phi.shape
    z = np.empty(G); sup = np.empty(k, dtype=np.int32)
    rh = np.empty(T + 1); gh = np.empty(max(T, 1))
    zp = None if z_prev is None else _f64(z_prev)
    z0a = None if z0 is None else _f64(z0)
    lib().oracle_iht_temporal(_p(Phi), _p(y), ctypes.c_int(m), ctypes.c_int(G), ctypes.c_int(k), ctypes.c_int(T),
                              ctypes.c_double(mu), ctypes.c_double(gamma), _p(zp), _p(z0a), _p(z), _p(sup), _p(rh), _p(gh))
    return IHTResult(z, sup, rh, gh[:T])


class NIHTResult(IHTResult):
    __slots__ = ("step_hist",)


def niht(Phi, y, k: int, T: int, mu_fallback: float) -> "NIHTResult":
    """IHT with the normalised step mu_t = ||g_S||^2 / ||Phi g_S||^2 (no line search); see cs_oracle.c."""
    Phi = _f32(Phi); y = _f64(y)
    m, G = Phi.shape
    z = np.empty(G); sup = np.empty(k, dtype=np.int32)
    rh = np.empty(T + 1); gh = np.empty(max(T, 1)); sh = np.empty(max(T, 1))
    lib().oracle_niht(_p(Phi), _p(y), ctypes.c_int(m), ctypes.c_int(G), ctypes.c_int(k), ctypes.c_int(T),
                      ctypes.c_double(mu_fallback), _p(z), _p(sup), _p(rh), _p(gh), _p(sh))
    r = NIHTResult(z, sup, rh, gh[:T])
    r.step_hist = sh[:T]
    return r


class OMPResult:
    __slots__ = ("z", "support", "order", "resid", "gap_hist")

    @property
    def min_gap(self) -> float:
        return float(self.gap_hist.min()) if self.gap_hist.size else float("inf")


def omp(Phi, y, k: int) -> OMPResult:
    """Orthogonal matching pursuit over the k-subsets of the G groups; see cs_oracle.c."""
    Phi = _f32(Phi); y = _f64(y)
    m, G = Phi.shape
    r = OMPResult()
    r.z = np.empty(G); r.support = np.empty(k, dtype=np.int32); r.order = np.empty(k, dtype=np.int32)
    r.gap_hist = np.empty(k)
    res = ctypes.c_double(0.0)
    lib().oracle_omp(_p(Phi), _p(y), ctypes.c_int(m), ctypes.c_int(G), ctypes.c_int(k), _p(r.z), _p(r.support),
                     _p(r.order), ctypes.byref(res), _p(r.gap_hist))
    r.resid = res.value
    return r


def srht(sign, rows, h) -> np.ndarray:
    """Subsampled randomized Hadamard sketch of one vector [d] or a batch [B, d] (d a power of two)."""
    sg = np.ascontiguousarray(np.asarray(sign), dtype=np.int8)
    rw = _i32(rows); h = _f64(h)
    d = h.shape[-1]; m = rw.shape[0]
    assert d & (d - 1) == 0 and sg.shape == (d,)
    flat = h.reshape(-1, d)
    y = np.empty((flat.shape[0], m))
    for i in range(flat.shape[0]):
        yi = np.empty(m)
        lib().oracle_srht(_p(sg), _p(rw), _p(np.ascontiguousarray(flat[i])), ctypes.c_int(m), ctypes.c_int(d), _p(yi))
        y[i] = yi
    return y.reshape(h.shape[:-1] + (m,))


def support_drift_ratio(prev, cur) -> np.ndarray:
    """Normalised support drift (Sec. 15 metric suite): D_t = |S_t symmetric-difference S_{t-1}| / |S_t union S_{t-1}|."""
    a = _i32(prev); b = _i32(cur)
    if a.ndim == 1:
        a, b = a[None, :], b[None, :]
    out = np.empty(a.shape[0])
    for t in range(a.shape[0]):
        sa, sb = set(a[t].tolist()), set(b[t].tolist())
        out[t] = len(sa ^ sb) / len(sa | sb)
    return out


def ffn(W_gate, W_up, Wd_t, group: int, h, support, return_act: bool = False):
    """SwiGLU FFN of one vector h [d] restricted to the groups in ``support``."""
    wg, dt = _weights(W_gate); wu, dt2 = _weights(W_up); wd, dt3 = _weights(Wd_t)
    assert dt == dt2 == dt3
    d = wg.shape[1]
    h = _f64(h); sup = _i32(support); k = sup.shape[0]
    out = np.empty(d); act = np.empty(k * group) if return_act else None
    lib().oracle_ffn(_p(wg), _p(wu), _p(wd), ctypes.c_int(dt), ctypes.c_int(d), ctypes.c_int(group),
                     _p(h), _p(sup), ctypes.c_int(k), _p(out), _p(act))
    return (out, act) if return_act else out


class LayerResult:
    __slots__ = ("x_out", "y", "z_full", "support", "z", "resid", "min_gap")


def layer_step(layer, x, *, group: int, k: int, T: int, mu: Optional[float] = None,
               rms_eps: float = 1e-5, add_residual: Optional[bool] = None,
               forced_support=None) -> LayerResult:
    """One measure -> recover -> execute step for a batch x [B, d].

    ``layer`` has attributes S, Phi, W_gate, W_up, Wd_t, gamma (None = no RMSNorm), mu.
    The residual add defaults to "on exactly when the layer has an RMSNorm gain".
    """
    S = _f32(layer.S); Phi = _f32(layer.Phi)
    wg, dt = _weights(layer.W_gate); wu, _ = _weights(layer.W_up); wd, _ = _weights(layer.Wd_t)
    gamma = None if layer.gamma is None else _f32(layer.gamma)
    if add_residual is None:
        add_residual = gamma is not None
    mu = layer.mu if mu is None else mu
    x = _f64(x); B, d = x.shape
    m, G = Phi.shape; d_ff = wg.shape[0]
    assert d_ff == G * group and S.shape == (m, d)
    forced = None if forced_support is None else _i32(forced_support)
    r = LayerResult()
    r.x_out = np.empty((B, d)); r.y = np.empty((B, m)); r.z_full = np.empty((B, G))
    r.support = np.empty((B, k), dtype=np.int32); r.z = np.empty((B, k))
    r.resid = np.empty(B); r.min_gap = np.empty(B)
    lib().oracle_layer_step(_p(S), _p(Phi), _p(wg), _p(wu), _p(wd), ctypes.c_int(dt), _p(gamma),
                            ctypes.c_double(rms_eps), ctypes.c_int(int(add_residual)),
                            ctypes.c_int(d), ctypes.c_int(d_ff), ctypes.c_int(group), ctypes.c_int(m),
                            ctypes.c_int(k), ctypes.c_int(T), ctypes.c_double(mu),
                            _p(x), ctypes.c_int(B), _p(forced),
                            _p(r.x_out), _p(r.y), _p(r.z_full), _p(r.support), _p(r.z), _p(r.resid),
                            _p(r.min_gap))
    return r


def prompt_support(S, Phi, H, k: int, T: int, mu: float):
    """(ybar [m], IHTResult) from the mean of the n per-token sketches of H [n, d]."""
    S = _f32(S); Phi = _f32(Phi); H = _f64(H)
    n, d = H.shape; m, G = Phi.shape
    ybar = np.empty(m); z = np.empty(G); sup = np.empty(k, dtype=np.int32)
    rh = np.empty(T + 1); gh = np.empty(max(T, 1))
    lib().oracle_prompt_support(_p(S), _p(Phi), _p(H), ctypes.c_int(n), ctypes.c_int(d), ctypes.c_int(m),
                                ctypes.c_int(G), ctypes.c_int(k), ctypes.c_int(T), ctypes.c_double(mu),
                                _p(ybar), _p(z), _p(sup), _p(rh), _p(gh))
    return ybar, IHTResult(z, sup, rh, gh[:T])


class BudgetResult:
    __slots__ = ("H", "x", "m")

    def __init__(self, H, x, m):
        self.H, self.x, self.m = H, x, m


def uds_budget(logits, m_base: float, gamma: float, m_min: int, m_max: int) -> BudgetResult:
    """Uncertainty-driven measurement budget (Sec. 8.1, "Uncertainty-Driven Adaptive Sensing").

    Per row of ``logits`` [B, V]: p = softmax(logits), H = -sum_v p_v log p_v (natural logarithm,
    0 log 0 = 0), x = m_base (1 + gamma H), m = clip(floor(x), m_min, m_max).  fp64 throughout; x is
    returned so that a comparison can tell how far the floor was from flipping.
    """
    L = _f64(logits)
    if L.ndim == 1:
        L = L[None, :]
    H = np.empty(L.shape[0]); x = np.empty(L.shape[0]); m = np.empty(L.shape[0], dtype=np.int32)
    for t in range(L.shape[0]):
        row = L[t]
        p = np.exp(row - row.max())
        p = p / p.sum()
        nz = p > 0
        H[t] = -(p[nz] * np.log(p[nz])).sum()
        x[t] = m_base * (1.0 + gamma * H[t])
        m[t] = int(min(max(np.floor(x[t]), m_min), m_max))
    return BudgetResult(H, x, m)


def support_drift(prev, cur) -> np.ndarray:
    """Support drift between consecutive decoding steps (Sec. 11): Delta_t = |S_t symmetric-difference
    S_{t-1}| per row of the two [B, k] index lists, by Python sets."""
    a = _i32(prev); b = _i32(cur)
    if a.ndim == 1:
        a, b = a[None, :], b[None, :]
    return np.array([len(set(a[t].tolist()) ^ set(b[t].tolist())) for t in range(a.shape[0])], dtype=np.int32)


def brute_force_support(Phi, y, k: int):
    """Best k-subset by exhaustive least squares: argmin_{|S|=k} min_c ||y - Phi_S c||.

    Returns (support ascending, coefficients, residual norm).  Subsets are
    visited in lexicographic order and a later subset wins only if strictly
    better, so ties go to the lexicographically first.  Tiny G only.
    """
    Phi = np.asarray(_f32(Phi), dtype=np.float64); y = _f64(y)
    G = Phi.shape[1]
    best = (None, None, np.inf)
    for sub in itertools.combinations(range(G), k):
        cols = Phi[:, sub]
        c, *_ = np.linalg.lstsq(cols, y, rcond=None)
        res = float(np.linalg.norm(y - cols @ c))
        if res < best[2]:
            best = (np.array(sub, dtype=np.int32), c, res)
    return best
