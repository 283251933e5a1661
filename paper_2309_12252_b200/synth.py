"""Seeded synthetic inputs for the DEER-GRU hot path.

This module holds NO arithmetic of the method itself (no cell, no Jacobian, no
scan): it only draws numbers.  It is the one module that both the CPU oracle's
tests and the CUDA path's tests / benchmark import, so that both sides consume
identical bytes.

Generator (documented so that any other implementation can reproduce it):

* ``fnv1a64(name)``: 64-bit FNV-1a hash of the UTF-8 stream name.
* ``key = mix(seed * GOLDEN + fnv1a64(name))`` with ``mix`` the SplitMix64
  finaliser and ``GOLDEN = 0x9E3779B97F4A7C15``.
* the i-th 64-bit word of a stream is ``mix(key + (i + 1) * GOLDEN)``
  (counter based: no state, any index can be produced on its own).
* uniform in (0, 1): ``((word >> 40) + 0.5) / 2**24`` (24 bits, never 0 or 1).
* normal: Box-Muller on words ``2i`` and ``2i + 1``:
  ``sqrt(-2 ln u0) * cos(2 pi u1)`` evaluated in float64, then cast.

The workloads mirror the shapes and value distributions of the paper's GRU
speed benchmark (Sec. 4.1: untrained GRU, random fp32 inputs, batch 16, zero
initial state) and of its long-series classification task (Sec. 4.3 /
App. B.3: 17,984 samples, 6 channels, 5 classes), for which seeded random
walks stand in for the dataset.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_MASK = (1 << 64) - 1


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def fnv1a64(name: str) -> int:
    h = 0xCBF29CE484222325
    for c in name.encode("utf-8"):
        h ^= c
        h = (h * 0x100000001B3) & _MASK
    return h


def stream_key(seed: int, name: str) -> np.uint64:
    k = (int(seed) * int(_GOLDEN) + fnv1a64(name)) & _MASK
    return _mix(np.array([k], dtype=np.uint64))[0]


def words(seed: int, name: str, count: int, offset: int = 0) -> np.ndarray:
    """``count`` raw 64-bit words of stream ``(seed, name)`` starting at ``offset``."""
    key = stream_key(seed, name)
    idx = np.arange(offset + 1, offset + count + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(key + idx * _GOLDEN)


def uniform01(seed: int, name: str, count: int, offset: int = 0) -> np.ndarray:
    """float64 uniforms in the open interval (0, 1), 24 random bits each."""
    w = words(seed, name, count, offset)
    return ((w >> np.uint64(40)).astype(np.float64) + 0.5) / float(1 << 24)


def uniform(seed: int, name: str, shape, lo: float, hi: float, dtype=np.float32) -> np.ndarray:
    n = int(np.prod(shape))
    out = np.empty(n, dtype=dtype)
    step = 1 << 22
    for s in range(0, n, step):
        c = min(step, n - s)
        out[s:s + c] = (lo + (hi - lo) * uniform01(seed, name, c, s)).astype(dtype)
    return out.reshape(shape)


def normal(seed: int, name: str, shape, dtype=np.float32) -> np.ndarray:
    """Standard normals by Box-Muller (one normal per pair of words)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=dtype)
    step = 1 << 21
    for s in range(0, n, step):
        c = min(step, n - s)
        u = uniform01(seed, name, 2 * c, 2 * s)
        r = np.sqrt(-2.0 * np.log(u[0::2]))
        out[s:s + c] = (r * np.cos(2.0 * math.pi * u[1::2])).astype(dtype)
    return out.reshape(shape)


def randint(seed: int, name: str, shape, high: int) -> np.ndarray:
    n = int(np.prod(shape))
    w = words(seed, name, n)
    return ((w >> np.uint64(33)) % np.uint64(high)).astype(np.int32).reshape(shape)


# ---------------------------------------------------------------------------
# GRU parameters and workloads
# ---------------------------------------------------------------------------

@dataclass
class GruParams:
    """Packed GRU parameters, gate order (r, z, n) along the leading 3n axis."""
    n: int
    m: int
    W_i: np.ndarray  # [3n, m]
    W_h: np.ndarray  # [3n, n]
    b_i: np.ndarray  # [3n]
    b_h: np.ndarray  # [3n]

    def astype(self, dtype) -> "GruParams":
        return GruParams(self.n, self.m, self.W_i.astype(dtype), self.W_h.astype(dtype),
                         self.b_i.astype(dtype), self.b_h.astype(dtype))


def gru_params(n: int, m: int, seed: int = 0, tag: str = "gru") -> GruParams:
    """Every entry ~ U(-1/sqrt(n), 1/sqrt(n)); streams W_i, W_h, b_i, b_h."""
    a = 1.0 / math.sqrt(n)
    return GruParams(
        n, m,
        uniform(seed, f"{tag}/W_i", (3 * n, m), -a, a),
        uniform(seed, f"{tag}/W_h", (3 * n, n), -a, a),
        uniform(seed, f"{tag}/b_i", (3 * n,), -a, a),
        uniform(seed, f"{tag}/b_h", (3 * n,), -a, a),
    )


def x_gaussian(B: int, T: int, m: int, seed: int = 0, tag: str = "x") -> np.ndarray:
    return normal(seed, tag, (B, T, m))


def x_sinusoid(B: int, T: int, m: int, seed: int = 0, tag: str = "xsin") -> np.ndarray:
    """x[b,t,c] = sin(omega[b,c] * t + phi[b,c]) + 0.1 * N(0,1), t = 0..T-1,
    omega ~ U(0.001, 0.1), phi ~ U(0, 2 pi), drawn per (sequence, channel)."""
    omega = uniform(seed, f"{tag}/omega", (B, 1, m), 0.001, 0.1, dtype=np.float64)
    phi = uniform(seed, f"{tag}/phi", (B, 1, m), 0.0, 2.0 * math.pi, dtype=np.float64)
    t = np.arange(T, dtype=np.float64).reshape(1, T, 1)
    eps = normal(seed, f"{tag}/eps", (B, T, m), dtype=np.float64)
    return (np.sin(omega * t + phi) + 0.1 * eps).astype(np.float32)


def x_random_walk(B: int, T: int, m: int, seed: int = 0, tag: str = "xwalk",
                  sigma: float = 0.05) -> np.ndarray:
    """Per-channel Gaussian random walk (step sigma), z-normalised per
    (sequence, channel) over T with the population standard deviation."""
    steps = normal(seed, tag, (B, T, m), dtype=np.float64) * sigma
    walk = np.cumsum(steps, axis=1)
    mu = walk.mean(axis=1, keepdims=True)
    sd = walk.std(axis=1, keepdims=True)
    return ((walk - mu) / sd).astype(np.float32)


@dataclass
class Workload:
    name: str
    B: int
    T: int
    n: int
    m: int
    params: GruParams
    x: np.ndarray   # [B, T, m] fp32
    y0: np.ndarray  # [B, n]    fp32


def config(idx: int, seed: int = 0, B: int | None = None, T: int | None = None) -> Workload:
    """The single-layer benchmark configurations 1..3 (1-based as listed in
    the benchmark definition); ``B``/``T`` may be reduced for quick checks."""
    if idx == 1:
        n, m, B0, T0, kind = 4, 2, 1, 1000, "gauss"
    elif idx == 2:
        n, m, B0, T0, kind = 8, 4, 16, 10000, "sin"
    elif idx == 3:
        n, m, B0, T0, kind = 32, 32, 16, 100000, "gauss"
    else:
        raise ValueError("config index must be 1, 2 or 3")
    B = B0 if B is None else B
    T = T0 if T is None else T
    p = gru_params(n, m, seed, tag=f"c{idx}/gru")
    if kind == "gauss":
        x = x_gaussian(B, T, m, seed, tag=f"c{idx}/x")
    else:
        x = x_sinusoid(B, T, m, seed, tag=f"c{idx}/x")
    return Workload(f"config{idx}", B, T, n, m, p, x, np.zeros((B, n), np.float32))


def sweep_point(n: int, T: int, B: int = 16, seed: int = 0) -> Workload:
    """Sweep configuration: m = n, x ~ N(0,1), y0 = 0."""
    p = gru_params(n, n, seed, tag=f"sweep{n}/gru")
    x = x_gaussian(B, T, n, seed, tag=f"sweep{n}/x")
    return Workload(f"sweep_n{n}_T{T}", B, T, n, n, p, x, np.zeros((B, n), np.float32))


@dataclass
class ClassifierWorkload:
    name: str
    B: int
    T: int
    layers: list          # [GruParams(n=64,m=6), GruParams(n=64,m=64)]
    W_o: np.ndarray       # [n_classes, n]
    b_o: np.ndarray       # [n_classes]
    x: np.ndarray         # [B, T, m]
    labels: np.ndarray    # [B] int32


def config4(seed: int = 0, B: int = 32, T: int = 17984, n: int = 64, m: int = 6,
            n_classes: int = 5) -> ClassifierWorkload:
    """Two stacked GRU layers, mean-pool over T, linear head, random labels."""
    l1 = gru_params(n, m, seed, tag="c4/gru1")
    l2 = gru_params(n, n, seed, tag="c4/gru2")
    a = 1.0 / math.sqrt(n)
    W_o = uniform(seed, "c4/W_o", (n_classes, n), -a, a)
    b_o = uniform(seed, "c4/b_o", (n_classes,), -a, a)
    x = x_random_walk(B, T, m, seed, tag="c4/x")
    labels = randint(seed, "c4/labels", (B,), n_classes)
    return ClassifierWorkload("config4", B, T, [l1, l2], W_o, b_o, x, labels)


@dataclass
class LstmParams:
    """Packed LSTM parameters, gate order (i, f, g, o) along the leading 4k axis; one bias vector."""
    k: int
    m: int
    W_i: np.ndarray  # [4k, m]
    W_h: np.ndarray  # [4k, k]
    b: np.ndarray    # [4k]


def lstm_params(k: int, m: int, seed: int = 0, tag: str = "lstm") -> LstmParams:
    """Every entry ~ U(-1/sqrt(k), 1/sqrt(k)); streams W_i, W_h, b."""
    a = 1.0 / math.sqrt(k)
    return LstmParams(k, m, uniform(seed, f"{tag}/W_i", (4 * k, m), -a, a), uniform(seed, f"{tag}/W_h", (4 * k, k), -a, a),
                      uniform(seed, f"{tag}/b", (4 * k,), -a, a))


def multihead_params(H: int, n: int, m: int, seed: int = 0, tag: str = "mh") -> list:
    """H independent parameter sets (one GRU head each), streams ``{tag}/head{h}/...``."""
    return [gru_params(n, m, seed, tag=f"{tag}/head{h}") for h in range(H)]


def multihead_strides(H: int, kinds: int = 8) -> np.ndarray:
    """Strides 2^0 .. 2^(kinds-1) assigned uniformly to the heads (App. B.4): head h gets 2^(h mod kinds)."""
    return (2 ** (np.arange(H) % kinds)).astype(np.int32)


def contractive_J(B: int, T: int, n: int, seed: int = 0, tag: str = "scanJ",
                  scale: float = 0.9) -> np.ndarray:
    """Random matrices with entries U(-s, s), s = scale / n, so that every
    row's absolute sum (hence the infinity norm) stays below ``scale``: a
    stand-in for GRU Jacobians of an untrained cell (contractive)."""
    s = scale / n
    return uniform(seed, tag, (B, T, n, n), -s, s)
