"""The generators of ``synth`` evaluated with torch integer ops, so that the large benchmark inputs
(gigabytes of Jacobians) can be drawn directly in device memory from the SAME documented streams.

No arithmetic of the method lives here: only the counter-based SplitMix64 words of ``synth`` (see the
generator description there), the 24-bit uniforms and the Box-Muller normals.  ``uniform`` is
bit-identical to ``synth.uniform`` (integer arithmetic plus one exactly rounded float64 multiply-add);
``normal`` agrees with ``synth.normal`` to the last float32 place or one unit of it (the float64
``log`` / ``cos`` of the two platforms may differ in their last bit before the cast).  A benchmark
point drawn here can therefore be re-drawn on the host and handed to the oracle.
"""
from __future__ import annotations

import math

import torch

from . import synth

_MASK64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Two's-complement int64 value of an unsigned 64-bit constant."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of int64 words (torch's >> is arithmetic)."""
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _uniform01(seed: int, name: str, count: int, offset: int, device) -> torch.Tensor:
    key = _s64(int(synth.stream_key(seed, name)))
    idx = torch.arange(offset + 1, offset + count + 1, dtype=torch.int64, device=device)
    w = _mix(idx * _GOLDEN + key)
    return (_lsr(w, 40).to(torch.float64) + 0.5) / float(1 << 24)


def uniform(seed: int, name: str, shape, lo: float, hi: float, device="cuda") -> torch.Tensor:
    """float32 tensor equal, bit for bit, to ``synth.uniform(seed, name, shape, lo, hi)``."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.float32, device=device)
    step = 1 << 24
    for s in range(0, n, step):
        c = min(step, n - s)
        out[s:s + c] = (lo + (hi - lo) * _uniform01(seed, name, c, s, device)).to(torch.float32)
    return out.reshape(shape)


def normal(seed: int, name: str, shape, device="cuda") -> torch.Tensor:
    """float32 standard normals from the stream of ``synth.normal(seed, name, shape)``."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.float32, device=device)
    step = 1 << 23
    for s in range(0, n, step):
        c = min(step, n - s)
        u = _uniform01(seed, name, 2 * c, 2 * s, device)
        r = torch.sqrt(-2.0 * torch.log(u[0::2]))
        out[s:s + c] = (r * torch.cos(2.0 * math.pi * u[1::2])).to(torch.float32)
    return out.reshape(shape)


def contractive_J(B: int, T: int, n: int, seed: int = 0, tag: str = "scanJ", scale: float = 0.9,
                  device="cuda") -> torch.Tensor:
    """``synth.contractive_J`` in device memory: entries U(-scale/n, scale/n)."""
    s = scale / n
    return uniform(seed, tag, (B, T, n, n), -s, s, device)
