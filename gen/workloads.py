"""Seeded synthetic FFN layers and hidden states for the five workloads.

Shapes follow Llama-2-7B / Llama-3-8B / Llama-2-13B feed-forward layers; the
values are synthetic (no trained weights exist here).  This module builds
*inputs only*: the probe A, the measurement matrix Phi, the products and
constants a caller of the library precomputes at model-load time
(S = Phi*A, the step size 1/||Phi||_2^2), the weights, and hidden states with a
planted group support.  It contains no sketch, recovery or FFN arithmetic.

Every tensor is a function of (seed, tensor id, layer, index) through
``gen.rng``; low-precision tensors are rounded to their storage type exactly
once, here, and both the CUDA library and the CPU oracle read those stored
values.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import torch

from . import rng

BASE_SEED = 260414156

# tensor ids (first component of the random stream)
T_A, T_PHI, T_WG, T_WU, T_WD, T_GAMMA, T_SUPP, T_COEF, T_NOISE, T_CBAR = range(1, 11)


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    index: int            # position in the workload list, offsets the seed
    d: int                # hidden size
    d_ff: int             # SwiGLU intermediate size
    group: int            # channels per group (b)
    m: int                # sketch rows
    k: int                # active groups per token
    T: int                # IHT iterations
    B: int                # decode batch (or prompt length when prompt=True)
    w_dtype: str          # "f32" | "bf16"
    sigma: float          # std of the noise added to the planted hidden state
    n_layers: int = 1
    rms: bool = False     # RMSNorm before the layer + residual add after it
    prompt: bool = False  # one shared support recovered from the mean prompt sketch
    rms_eps: float = 1e-5

    @property
    def G(self) -> int:
        return self.d_ff // self.group

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    def with_(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, Config] = {
    "tiny_f32": Config("tiny_f32", 0, d=256, d_ff=1024, group=64, m=8, k=4, T=10, B=4,
                       w_dtype="f32", sigma=0.01),
    "l2_7b_b1": Config("l2_7b_b1", 1, d=4096, d_ff=11008, group=128, m=32, k=22, T=20, B=1,
                       w_dtype="bf16", sigma=0.05),
    "l2_7b_b64": Config("l2_7b_b64", 2, d=4096, d_ff=11008, group=128, m=32, k=22, T=20, B=64,
                        w_dtype="bf16", sigma=0.05),
    "l3_8b_stack": Config("l3_8b_stack", 3, d=4096, d_ff=14336, group=128, m=48, k=28, T=20, B=32,
                          w_dtype="bf16", sigma=0.05, n_layers=32, rms=True),
    "l2_13b_prompt": Config("l2_13b_prompt", 4, d=5120, d_ff=13824, group=128, m=64, k=27, T=20,
                            B=2048, w_dtype="bf16", sigma=0.05, prompt=True),
}
PROMPT_K_SWEEP = (11, 27, 54)  # 10 / 25 / 50 % of G = 108


def _torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


@dataclasses.dataclass
class Layer:
    A: torch.Tensor          # [G, d] float64, unit-norm rows (CPU; only used to plant h)
    Phi: torch.Tensor        # [m, G] float32
    S: torch.Tensor          # [m, d] float32 = Phi * A (float64 product, rounded once)
    mu: float                # step size 1 / ||Phi||_2^2, a float32 value
    W_gate: torch.Tensor     # [d_ff, d]
    W_up: torch.Tensor       # [d_ff, d]
    Wd_t: torch.Tensor       # [d_ff, d] = W_down transposed
    gamma: Optional[torch.Tensor]  # [d] float32 RMSNorm gain, or None

    def to(self, device) -> "Layer":
        mv = lambda t: None if t is None else t.to(device)
        return Layer(self.A, mv(self.Phi), mv(self.S), self.mu, mv(self.W_gate), mv(self.W_up),
                     mv(self.Wd_t), mv(self.gamma))


def spectral_step(Phi: torch.Tensor) -> float:
    """1 / ||Phi||_2^2 of the stored float32 Phi, rounded to float32."""
    smax = torch.linalg.svdvals(Phi.detach().to("cpu", torch.float64))[0].item()
    return float(torch.tensor(1.0 / (smax * smax), dtype=torch.float32).item())


def make_probe(cfg: Config, layer: int = 0) -> torch.Tensor:
    """Probe A [G, d]: N(0,1) rows scaled to unit length (float64, CPU)."""
    A = rng.normal(cfg.seed, (T_A, layer), (cfg.G, cfg.d))
    return A / A.norm(dim=1, keepdim=True)


def make_layer(cfg: Config, layer: int = 0, device="cpu", literal_mu: Optional[float] = None) -> Layer:
    """All parameters of one layer; the large weight tensors are built on ``device``."""
    A = make_probe(cfg, layer)
    Phi = rng.normal(cfg.seed, (T_PHI, layer), (cfg.m, cfg.G), dtype=torch.float32,
                     scale=1.0 / math.sqrt(cfg.m))
    S = (Phi.to(torch.float64) @ A).to(torch.float32)
    mu = spectral_step(Phi) if literal_mu is None else float(literal_mu)
    wd = _torch_dtype(cfg.w_dtype)
    shape = (cfg.d_ff, cfg.d)
    Wg = rng.normal(cfg.seed, (T_WG, layer), shape, device, wd, 1.0 / math.sqrt(cfg.d))
    Wu = rng.normal(cfg.seed, (T_WU, layer), shape, device, wd, 1.0 / math.sqrt(cfg.d))
    Wdt = rng.normal(cfg.seed, (T_WD, layer), shape, device, wd, 1.0 / math.sqrt(cfg.d_ff))
    gamma = None
    if cfg.rms:
        gamma = (1.0 + 0.1 * rng.normal(cfg.seed, (T_GAMMA, layer), cfg.d)).to(torch.float32).to(device)
    return Layer(A, Phi.to(device), S.to(device), mu, Wg, Wu, Wdt, gamma)


@dataclasses.dataclass
class Tokens:
    planted: torch.Tensor    # [B, k] int32 (or [1, k] for a prompt), ascending
    h: torch.Tensor          # [B, d] float32 (bfloat16 for a prompt), CPU


def make_tokens(cfg: Config, A: torch.Tensor, batch: int = 0, B: Optional[int] = None) -> Tokens:
    """Hidden states h = sum_{g in planted} c_g A_g + N(0, sigma^2).

    Decode workloads: an independent uniform k-subset and c_g ~ N(0,1) per token.
    Prompt workload: one subset for the whole prompt; per-token coefficients
    c_{g,i} = cbar_g + 0.25 N(0,1) around a per-prompt mean cbar_g ~ N(0,1)
    whose magnitude is floored at 0.5 (so the mean sketch carries the support).
    """
    B = cfg.B if B is None else B
    G, k, d = cfg.G, cfg.k, cfg.d
    if cfg.prompt:
        planted = rng.k_subset(cfg.seed, (T_SUPP, batch), G, k, rows=1)
        cbar = rng.normal(cfg.seed, (T_CBAR, batch), k)
        cbar = torch.where(cbar.abs() < 0.5, torch.where(cbar < 0, -0.5, 0.5).to(cbar.dtype), cbar)
        c = cbar[None, :] + 0.25 * rng.normal(cfg.seed, (T_COEF, batch), (B, k))
        rows = A[planted[0].long()]                      # [k, d]
        h = c @ rows
    else:
        planted = rng.k_subset(cfg.seed, (T_SUPP, batch), G, k, rows=B)
        c = rng.normal(cfg.seed, (T_COEF, batch), (B, k))
        h = torch.einsum("bk,bkd->bd", c, A[planted.long()])
    h = h + cfg.sigma * rng.normal(cfg.seed, (T_NOISE, batch), (B, d))
    h = h.to(torch.bfloat16 if cfg.prompt else torch.float32)
    return Tokens(planted, h)
