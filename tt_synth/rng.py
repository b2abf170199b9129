"""Counter-based random numbers: splitmix64 of (seed, tensor id, element index).

Every value is a pure function of its coordinates, so any sub-range of any tensor can be
generated independently and in any order (vectorised here with numpy uint64 arithmetic).
splitmix64 is the public-domain finaliser by Steele, Lea and Flood ("Fast splittable
pseudorandom number generators", OOPSLA 2014): z += 0x9E3779B97F4A7C15; two xor-shift
multiply rounds; final xor-shift.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_TENSOR_STRIDE = np.uint64(0xD1B54A32D192ED03)
_SEED_STRIDE = np.uint64(0x8CB92BA72F3D8DD7)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """One splitmix64 output per 64-bit input state (vectorised, wraps modulo 2**64)."""
    with np.errstate(over="ignore"):
        z = np.asarray(x, dtype=np.uint64) + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _counters(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        base = (np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _SEED_STRIDE
                + np.uint64(tensor_id & 0xFFFFFFFFFFFFFFFF) * _TENSOR_STRIDE)
        idx = np.arange(start, start + count, dtype=np.uint64)
        # two rounds so that nearby (seed, tensor, index) triples decorrelate
        return splitmix64(splitmix64(base) + idx)


def raw_u64(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    return _counters(seed, tensor_id, start, count)


def uniform01(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """float64 uniform in [0, 1) with 53 random bits."""
    u = _counters(seed, tensor_id, start, count)
    return (u >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def normal(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """float64 standard normal by Box-Muller on counter pairs (2i, 2i+1)."""
    u = uniform01(seed, tensor_id, 2 * count, 2 * start)
    u1 = 1.0 - u[0::2]          # (0, 1]
    u2 = u[1::2]
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
