"""Seeded synthetic inputs for the WCC layer: feature maps and 1x1 weights.

This module only produces bytes.  It holds none of the layer's arithmetic
(no Haar step, no ranking, no quantizer, no contraction) and is the one
module that both the CUDA path's tests and the CPU oracle's tests may use.

Feature maps stand in for CNN activations after a ReLU: every channel is
``max(v, 0) + 0.05 * eps`` with ``v`` a sum of ``S`` random 2-D sinusoids
(frequencies uniform in ``[0, F]`` cycles per image, uniform phases,
standard-normal amplitudes) and ``eps`` iid standard normal.  Weights are
``N(0, 1/Cin)``.  Everything is computed in float64 from a counter-based
generator (the SplitMix64 output function applied to ``key + (i+1)*gamma``,
Steele, Lea & Flood 2014), so a value depends only on (seed, stream id,
element index) and never on a library's generator version.  The result is
rounded once to fp32, or to bf16 by round-to-nearest-even, and both sides
read those same bytes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# stream ids (which tensor a counter belongs to)
STREAM_FX, STREAM_FY, STREAM_PHASE, STREAM_AMP, STREAM_NOISE, STREAM_WEIGHT = 1, 2, 3, 4, 5, 6


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on an array of uint64."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.array([(seed & 0xFFFFFFFF) | ((stream & 0xFFFFFFFF) << 32)], dtype=np.uint64)
        return _mix(k * _GAMMA + _GAMMA)[0]


def raw_u64(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """``count`` 64-bit words of stream ``stream`` beginning at counter ``start``."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + 1 + count, dtype=np.uint64)
        return _mix(_key(seed, stream) + ctr * _GAMMA)


def uniform01(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """float64 uniform in [0, 1) with 53 random bits."""
    return (raw_u64(seed, stream, start, count) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def normal(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """float64 standard normal by Box-Muller; element i uses counters 2i, 2i+1."""
    u = uniform01(seed, stream, 2 * start, 2 * count)
    u1 = 1.0 - u[0::2]          # (0, 1]
    u2 = u[1::2]
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = b + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def feature_map(seed: int, N: int, C: int, H: int, W: int, n_sin: int, fmax: float,
                noise_std: float = 0.05) -> np.ndarray:
    """float64 [N][C][H][W] smooth-sinusoid + noise ReLU maps."""
    planes = N * C
    fx = uniform01(seed, STREAM_FX, 0, planes * n_sin).reshape(planes, n_sin) * fmax
    fy = uniform01(seed, STREAM_FY, 0, planes * n_sin).reshape(planes, n_sin) * fmax
    ph = uniform01(seed, STREAM_PHASE, 0, planes * n_sin).reshape(planes, n_sin) * (2.0 * math.pi)
    am = normal(seed, STREAM_AMP, 0, planes * n_sin).reshape(planes, n_sin)
    col = np.arange(W, dtype=np.float64) / W
    row = np.arange(H, dtype=np.float64) / H
    out = np.empty((planes, H, W), dtype=np.float64)
    step = max(1, (1 << 22) // (H * W))          # planes per slab, bounds the temporaries
    for p0 in range(0, planes, step):
        p1 = min(planes, p0 + step)
        A = 2.0 * math.pi * fx[p0:p1, :, None] * col[None, None, :] + ph[p0:p1, :, None]   # [p][s][W]
        B = 2.0 * math.pi * fy[p0:p1, :, None] * row[None, None, :]                         # [p][s][H]
        a = am[p0:p1, :, None]
        # sin(A + B) = sin A cos B + cos A sin B, summed over the sinusoids
        left = np.concatenate([(a * np.cos(B)).transpose(0, 2, 1), (a * np.sin(B)).transpose(0, 2, 1)], axis=2)
        right = np.concatenate([np.sin(A), np.cos(A)], axis=1)
        v = np.matmul(left, right)                                                         # [p][H][W]
        eps = normal(seed, STREAM_NOISE, p0 * H * W, (p1 - p0) * H * W).reshape(p1 - p0, H, W)
        out[p0:p1] = np.maximum(v, 0.0) + noise_std * eps
    return out.reshape(N, C, H, W)


def weights(seed: int, Cout: int, Cin: int, stream: int = STREAM_WEIGHT) -> np.ndarray:
    """fp32 [Cout][Cin] drawn N(0, 1/Cin)."""
    w = normal(seed, stream, 0, Cout * Cin).reshape(Cout, Cin) / math.sqrt(Cin)
    return w.astype(np.float32)


@dataclass
class Workload:
    """One WCC layer call: shapes, parameters and the bytes both sides read."""
    name: str
    N: int
    Cin: int
    Cout: int
    H: int
    W: int
    levels: int
    k: int
    bits: int
    dtype: str                      # "f32" or "bf16"
    x: np.ndarray = field(repr=False, default=None)      # fp32 array, or uint16 bf16 bit patterns
    Wt: np.ndarray = field(repr=False, default=None)     # fp32 [Cout][Cin]

    @property
    def P(self) -> int:
        return self.H * self.W

    def x_f32(self) -> np.ndarray:
        """The activations widened exactly to fp32."""
        return bf16_bits_to_f32(self.x) if self.dtype == "bf16" else self.x


def keep_count(gamma: float, P: int) -> int:
    """k = ceil(gamma * P), the number of kept positions per image."""
    return int(math.ceil(gamma * P - 1e-9))


# name: (N, Cin, Cout, H, W, dtype, levels, gamma, bits, n_sin, fmax)
CONFIGS = {
    "C1": (1, 32, 32, 64, 64, "f32", 2, 0.25, 8, 8, 4.0),
    "C2": (4, 144, 24, 128, 256, "bf16", 3, 0.5, 8, 16, 8.0),
    "C3": (2, 24, 144, 256, 512, "bf16", 3, 0.25, 8, 16, 8.0),
    "C3u": (2, 24, 144, 256, 512, "bf16", 3, 0.25, 0, 16, 8.0),
    "C4": (12, 64, 64, 96, 320, "f32", 2, 0.125, 8, 16, 8.0),
    "C4b": (12, 64, 64, 96, 320, "f32", 2, 0.0625, 8, 16, 8.0),
    "C5a": (2, 32, 192, 256, 512, "bf16", 3, 0.25, 8, 16, 8.0),
    "C5b": (2, 192, 32, 256, 512, "bf16", 3, 0.25, 8, 16, 8.0),
}


def make(name: str, seed: int = 0, **override) -> Workload:
    """Build a named workload (see ``CONFIGS``); keyword overrides replace table entries."""
    N, Cin, Cout, H, W, dtype, levels, gamma, bits, n_sin, fmax = CONFIGS[name]
    p = dict(N=N, Cin=Cin, Cout=Cout, H=H, W=W, dtype=dtype, levels=levels, gamma=gamma,
             bits=bits, n_sin=n_sin, fmax=fmax)
    p.update(override)
    return custom(name=name, seed=seed, **p)


def custom(name: str, seed: int, N: int, Cin: int, Cout: int, H: int, W: int, dtype: str,
           levels: int, gamma: float, bits: int, n_sin: int = 8, fmax: float = 4.0,
           k: int | None = None) -> Workload:
    xd = feature_map(seed, N, Cin, H, W, n_sin, fmax)
    x32 = xd.astype(np.float32)
    x = f32_to_bf16_bits(x32) if dtype == "bf16" else x32
    Wt = weights(seed, Cout, Cin)
    kk = keep_count(gamma, H * W) if k is None else k
    return Workload(name=name, N=N, Cin=Cin, Cout=Cout, H=H, W=W, levels=levels, k=kk, bits=bits,
                    dtype=dtype, x=x, Wt=Wt)
