"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This module holds no layer arithmetic: it only produces reproducible NCHW
arrays (activations, filters, biases) and, in `synth.configs`, the plain
descriptions of the workloads (shapes and layer lists).  Every value is a pure
function of (seed, tensor id, flat index), so any slice of a tensor can be
regenerated on its own and the same bytes reach both implementations.

Generator: the SplitMix64 finaliser (Steele, Lea, Flood 2014) applied to a
64-bit counter built from seed, tensor id and element index; the top 24 bits
give a uniform in [0, 1) that is exactly representable in float32.  Normal
deviates use the Box-Muller transform on two such uniforms.
"""
from __future__ import annotations

import numpy as np

DEFAULT_SEED = 20230304

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = z + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _counter(seed: int, tensor_id: int, start: int, count: int, lane: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(seed & 0xFFFFFFFF) << 32 | (tensor_id & 0xFFFFFFFF)], dtype=np.uint64))[0]
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _splitmix64(key ^ (idx * np.uint64(2) + np.uint64(lane)))


def unit_uniform(seed: int, tensor_id: int, count: int, start: int = 0, lane: int = 0) -> np.ndarray:
    """`count` float64 uniforms in [0,1) on a 2^-24 grid, for flat indices start..start+count."""
    bits = _counter(seed, tensor_id, start, count, lane)
    return (bits >> np.uint64(40)).astype(np.float64) * (1.0 / 16777216.0)


def uniform(shape, lo: float, hi: float, tensor_id: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """float32 array of `shape`, uniform on [lo, hi)."""
    n = int(np.prod(shape))
    u = unit_uniform(seed, tensor_id, n)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(shape, mean: float, std: float, tensor_id: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """float32 array of `shape`, normal(mean, std^2) by Box-Muller on two uniforms per element."""
    n = int(np.prod(shape))
    u1 = unit_uniform(seed, tensor_id, n, lane=0)
    u2 = unit_uniform(seed, tensor_id, n, lane=1)
    u1 = 1.0 - u1  # (0, 1]: keeps the logarithm finite
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def he_normal(shape, fan_in: int, tensor_id: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """He initialisation: normal(0, 2 / fan_in)."""
    return normal(shape, 0.0, float(np.sqrt(2.0 / fan_in)), tensor_id, seed)
