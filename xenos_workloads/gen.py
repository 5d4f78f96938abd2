"""Seeded synthetic tensors shared by the CPU oracle's tests and the CUDA library's tests.

Holds no operator arithmetic: only a counter-based generator.  Element ``i`` of tensor ``t``
under seed ``s`` is a pure function of (s, t, i), so tensors can be produced in any order, in
pieces, and identically on every machine.

Generator: the splitmix64 output function applied to a 64-bit counter built from
(seed, tensor id, element index).  Uniforms take the top 24 bits (exact in fp32); normals are
Box-Muller over two independent uniforms.
"""
from __future__ import annotations

import numpy as np

DEFAULT_SEED = 20230200

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z + _GOLD) & _M64
        z = ((z ^ (z >> np.uint64(30))) * _C1) & _M64
        z = ((z ^ (z >> np.uint64(27))) * _C2) & _M64
        return z ^ (z >> np.uint64(31))


def _bits(seed: int, tensor_id: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    with np.errstate(over="ignore"):
        key = _mix(np.array([(seed * 0x632BE59BD9B4E019 + tensor_id * 0xD1342543DE82EF95
                              + stream * 0x2545F4914F6CDD1D) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0]
        idx = np.arange(start, start + n, dtype=np.uint64)
        return _mix((idx * _GOLD + key) & _M64)


def _unit(seed, tensor_id, stream, n, start=0) -> np.ndarray:
    """Uniform on the open interval (0, 1): (top 24 bits + 0.5) / 2^24, in float64."""
    b = _bits(seed, tensor_id, stream, n, start) >> np.uint64(40)
    return (b.astype(np.float64) + 0.5) / float(1 << 24)


def uniform(seed: int, tensor_id: int, shape, lo: float, hi: float) -> np.ndarray:
    n = int(np.prod(shape))
    u = _unit(seed, tensor_id, 0, n)
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(seed: int, tensor_id: int, shape, mean: float, std: float) -> np.ndarray:
    n = int(np.prod(shape))
    u1 = _unit(seed, tensor_id, 1, n)
    u2 = _unit(seed, tensor_id, 2, n)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def index_valued(shape, modulus: int = 251) -> np.ndarray:
    """x[i] = i mod a small prime: makes a layout or index mistake show up as a wrong value."""
    n = int(np.prod(shape))
    return (np.arange(n, dtype=np.int64) % modulus).astype(np.float32).reshape(shape)
