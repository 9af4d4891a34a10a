"""Seeded synthetic tensors.  Holds no arithmetic of the method.

Every value is a pure function of (seed, tensor_id, flat index) through a 64-bit
counter-based mixer, so the same bytes can be regenerated anywhere, in any order,
and fed to the CUDA path and to the CPU oracle alike.
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser, vectorised over uint64."""
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _bits(seed: int, tensor_id: int, n: int, stream: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        base = _mix(np.array([(seed * 0x100000001B3 + tensor_id * 0x9E3779B1 + stream) & 0xFFFFFFFFFFFFFFFF],
                             dtype=np.uint64))[0]
        idx = np.arange(n, dtype=np.uint64)
        return _mix(idx ^ base)


def _unit(seed, tensor_id, n, stream=0) -> np.ndarray:
    """Uniform in [0, 1) with 53 random bits."""
    return (_bits(seed, tensor_id, n, stream) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def uniform(shape, seed: int, tensor_id: int, lo=-1.0, hi=1.0) -> np.ndarray:
    n = int(np.prod(shape)) if len(shape) else 1
    return (lo + (hi - lo) * _unit(seed, tensor_id, n)).astype(np.float32).reshape(shape)


def normal(shape, seed: int, tensor_id: int, std=1.0, mean=0.0) -> np.ndarray:
    n = int(np.prod(shape)) if len(shape) else 1
    u1 = 1.0 - _unit(seed, tensor_id, n, stream=1)          # (0, 1]
    u2 = _unit(seed, tensor_id, n, stream=2)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)
