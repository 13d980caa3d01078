"""Seeded synthetic tensors for tests and benchmarks.

This module is the only code the CUDA path's harness and the CPU oracle's
harness have in common.  It holds no arithmetic of the ternarization method:
it only draws numbers and rounds them to the storage types (fp32 master
weights, bf16 activations).

Generator definition (counter based, so any element can be drawn alone):

  key(seed, name)  = mix64(seed * GOLDEN + fnv1a64(name))
  bits(key, i)     = mix64(key + (i + 1) * GOLDEN)          (SplitMix64 output)
  u(key, i)        = (bits >> 11) * 2**-53                   in [0, 1)
  uniform[-1, 1)   = 2u - 1
  normal           = Box-Muller on the pair (u(2j), u(2j+1)):
                       r = sqrt(-2 ln(1 - u0)),  z(2j) = r cos(2 pi u1),
                       z(2j+1) = r sin(2 pi u1)
  laplace(0, 1)    = -sign(u - 1/2) * ln(1 - 2 |u - 1/2|)

All math is fp64 (numpy); the result is rounded to nearest-even to fp32, and
for activations once more to nearest-even to bf16 (stored as uint16).
"""
from __future__ import annotations

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix64(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _fnv1a64(name: str) -> int:
    h = 0xCBF29CE484222325
    for b in name.encode("utf-8"):
        h = ((h ^ b) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def stream_key(seed: int, name: str) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * GOLDEN + np.uint64(_fnv1a64(name))
        return _mix64(np.array([k], dtype=np.uint64))[0]


def _uniform01(key: np.uint64, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        i = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        bits = _mix64(key + i * GOLDEN)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def _draw_chunk(key, dist: str, start: int, count: int) -> np.ndarray:
    """fp64 samples for elements [start, start+count); start must be even."""
    if dist == "uniform01":
        return _uniform01(key, start, count)
    if dist == "uniform":
        return 2.0 * _uniform01(key, start, count) - 1.0
    if dist == "laplace":
        u = _uniform01(key, start, count) - 0.5
        return -np.sign(u) * np.log1p(-2.0 * np.abs(u))
    if dist == "normal":
        m = count + (count & 1)
        u = _uniform01(key, start, m)
        r = np.sqrt(-2.0 * np.log1p(-u[0::2]))
        t = (2.0 * np.pi) * u[1::2]
        z = np.empty(m, dtype=np.float64)
        z[0::2] = r * np.cos(t)
        z[1::2] = r * np.sin(t)
        return z[:count]
    raise ValueError(f"unknown distribution {dist!r}")


def draw(seed: int, name: str, n: int, dist: str, mean: float = 0.0,
         std: float = 1.0) -> np.ndarray:
    """n fp32 samples of `dist` in {"normal", "laplace", "uniform", "uniform01"},
    scaled as mean + std * sample (in fp64) before rounding to fp32."""
    key = stream_key(seed, name)
    out = np.empty(n, dtype=np.float32)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        x = _draw_chunk(key, dist, s, c)
        if std != 1.0:
            x = x * std
        if mean != 0.0:
            x = x + mean
        out[s:s + c] = x.astype(np.float32)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = (b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    w = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return w.view(np.float32).astype(np.float64)


def draw_bf16(seed: int, name: str, n: int, dist: str, mean: float = 0.0,
              std: float = 1.0) -> np.ndarray:
    """n bf16 samples as uint16 bit patterns."""
    return f32_to_bf16_bits(draw(seed, name, n, dist, mean, std))


def he_normal(seed: int, name: str, rows: int, fan_in: int) -> np.ndarray:
    """fp32 [rows, fan_in] master weights, N(0, 2/fan_in) (variance)."""
    w = draw(seed, name, rows * fan_in, "normal", 0.0, float(np.sqrt(2.0 / fan_in)))
    return w.reshape(rows, fan_in)
