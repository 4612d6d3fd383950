"""Counter-based seeded random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index): the 64-bit word
``mix64(key(seed, stream) + index * GOLDEN)`` where ``mix64`` is the
splitmix64 output function (Steele, Lea, Flood 2014).  Normals come from one
word per value by Box-Muller on its two 32-bit halves.  Nothing here knows
about the method (sketch, recovery, FFN): this module only makes numbers.

The arithmetic runs in torch int64/float64 tensors so the large weight
tensors can be produced directly in device memory; integer steps are exact
on every device, the float64 log/cos may differ in the last place between
devices, which is why a tensor is generated once and the same stored values
are handed to every consumer.
"""
from __future__ import annotations

import math
from typing import Iterable, Sequence

import torch

_MASK64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

_CHUNK = 1 << 24  # elements per pass: bounds the int64/float64 temporaries


def _signed(v: int) -> int:
    """Two's-complement int64 value of an unsigned 64-bit constant."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def mix64_int(x: int) -> int:
    """splitmix64 output function on a Python integer (reference form)."""
    x &= _MASK64
    x = ((x ^ (x >> 30)) * _M1) & _MASK64
    x = ((x ^ (x >> 27)) * _M2) & _MASK64
    return x ^ (x >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _signed(_M1)
    x = (x ^ _lsr(x, 27)) * _signed(_M2)
    return x ^ _lsr(x, 31)


def stream_key(seed: int, stream: Sequence[int] | int) -> int:
    """Fold a seed and a tuple of small integers into one 64-bit key."""
    if isinstance(stream, int):
        stream = (stream,)
    k = mix64_int(seed + GOLDEN)
    for s in stream:
        k = mix64_int(k ^ mix64_int((int(s) + 1) * GOLDEN))
    return k


def bits(seed: int, stream, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n 64-bit words (as int64) for indices offset .. offset+n-1."""
    key = stream_key(seed, stream)
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    return _mix64(idx * _signed(GOLDEN) + _signed(key))


def word_int(seed: int, stream, index: int) -> int:
    """The same word as ``bits`` computed with Python integers (for tests)."""
    key = stream_key(seed, stream)
    return mix64_int(key + index * GOLDEN)


def uniform(seed: int, stream, n: int, device="cpu") -> torch.Tensor:
    """n float64 uniforms in (0, 1): the top 53 bits of each word, centred."""
    w = bits(seed, stream, n, device)
    return (_lsr(w, 11).to(torch.float64) + 0.5) * (1.0 / (1 << 53))


def _normal_chunk(seed, stream, n, device, offset) -> torch.Tensor:
    w = bits(seed, stream, n, device, offset)
    hi = _lsr(w, 32).to(torch.float64)
    lo = (w & 0xFFFFFFFF).to(torch.float64)
    u1 = (hi + 0.5) * (1.0 / (1 << 32))
    u2 = (lo + 0.5) * (1.0 / (1 << 32))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def normal(seed: int, stream, shape: Iterable[int] | int, device="cpu",
           dtype=torch.float64, scale: float = 1.0) -> torch.Tensor:
    """N(0, scale^2) values of the given shape, rounded once to ``dtype``.

    Values are drawn in float64 and converted with round-to-nearest-even,
    which is the only rounding the stored tensor ever sees.
    """
    if isinstance(shape, int):
        shape = (shape,)
    shape = tuple(int(s) for s in shape)
    n = 1
    for s in shape:
        n *= s
    out = torch.empty(n, dtype=dtype, device=device)
    for off in range(0, n, _CHUNK):
        c = min(_CHUNK, n - off)
        v = _normal_chunk(seed, stream, c, device, off)
        if scale != 1.0:
            v = v * scale
        out[off:off + c] = v.to(dtype)
    return out.reshape(shape)


def k_subset(seed: int, stream, G: int, k: int, rows: int = 1, device="cpu") -> torch.Tensor:
    """``rows`` independent uniform k-subsets of {0..G-1}, each ascending.

    A subset is the positions of the k smallest of G distinct random words.
    """
    w = bits(seed, stream, rows * G, device).reshape(rows, G)
    # order words as unsigned: flip the sign bit so int64 ordering matches
    order = torch.argsort(w ^ _signed(1 << 63), dim=1, stable=True)
    return torch.sort(order[:, :k], dim=1).values.to(torch.int32)
