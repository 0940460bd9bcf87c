"""Counter-based seeded random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index), so arrays of any size can be
regenerated bit-for-bit on any machine and any numpy version.  The mixer is the
published splitmix64 finaliser (Steele, Lea, Flood 2014) applied to a counter.

This module holds no arithmetic of the sparse-convolution method: it only makes inputs.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 states."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def bits64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n pseudo-random uint64 words for (seed, stream), starting at counter `offset`."""
    with np.errstate(over="ignore"):
        key = _mix(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)]) * _GOLDEN
                   + np.uint64(stream & 0xFFFFFFFFFFFFFFFF))[0]
        ctr = np.arange(offset, offset + n, dtype=np.uint64)
        return _mix(key + (ctr + np.uint64(1)) * _GOLDEN)


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    """float32 uniforms on the grid k * 2^-24, k in [0, 2^24): exactly representable, < 1."""
    b = bits64(seed, stream, n)
    return ((b >> np.uint64(40)).astype(np.float32)) * np.float32(2.0 ** -24)


def uniform01_f64(seed: int, stream: int, n: int) -> np.ndarray:
    """float64 uniforms on the open-closed interval (0, 1] with 53 random bits."""
    b = bits64(seed, stream, n)
    return ((b >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)


def normal(seed: int, stream: int, n: int, sigma: float = 1.0) -> np.ndarray:
    """float64 N(0, sigma^2) by Box-Muller on two independent counter streams."""
    m = (n + 1) // 2
    u1 = uniform01_f64(seed, 2 * stream + 0x1000, m)
    u2 = uniform01_f64(seed, 2 * stream + 0x1001, m)
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * m, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n] * sigma


def permutation(seed: int, stream: int, n: int) -> np.ndarray:
    """A seeded permutation of range(n): stable argsort of n random 64-bit keys."""
    return np.argsort(bits64(seed, stream, n), kind="stable")


def to_bf16_bits(x):
    """float32 array -> bfloat16 bit patterns (uint16), round to nearest, ties to even; NaNs stay NaNs.
    Input preparation only: the values a bfloat16 workload feeds to both sides."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    return np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), rounded).astype(np.uint16)
