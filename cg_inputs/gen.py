"""Seeded synthetic inputs: an index-pure counter-based generator.

This module serves both the CPU oracle's tests and the CUDA path's tests/benchmark.  It holds
none of the method's arithmetic -- only random numbers and their rounding to the storage dtype.

Element ``idx`` (row-major logical index, whatever the storage order) of tensor ``tensor_id``
under ``seed`` is a pure function of (seed, tensor_id, idx):

    key      = mix(mix(seed) + tensor_id)
    x_j(idx) = mix(key + 2*idx + j),  j in {0, 1}          (64-bit, wrapping)
    u0 = (x_0 >> 11) * 2^-53 in [0,1)       u0' = ((x_0 >> 11) + 1) * 2^-53 in (0,1]
    u1 = (x_1 >> 11) * 2^-53
    uniform[-1,1):  2*u0 - 1
    normal(0, s):   s * sqrt(-2 ln u0') * cos(2 pi u1)      (s is a standard deviation)

``mix`` is the SplitMix64 output function.  Values are produced in fp64 and rounded once to the
storage dtype (bf16: round-to-nearest-even of the fp32 value; fp32: numpy's cast).
bf16 tensors are returned as ``uint16`` bit patterns.
"""
from __future__ import annotations

import numpy as np

TENSOR_A, TENSOR_B, TENSOR_BIAS, TENSOR_R = 1, 2, 3, 4
TENSOR_ROW_SCALE, TENSOR_COL_SCALE = 5, 6

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_CHUNK = 1 << 20


def _mix(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on uint64 arrays (wrapping arithmetic)."""
    z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([seed], dtype=np.uint64))
        k = _mix(k + np.uint64(tensor_id))
    return k[0]


def _raw(seed: int, tensor_id: int, idx: np.ndarray):
    with np.errstate(over="ignore"):
        base = _key(seed, tensor_id) + np.uint64(2) * idx.astype(np.uint64)
        return _mix(base), _mix(base + np.uint64(1))


def values_f64(seed: int, tensor_id: int, idx: np.ndarray, dist: str, scale: float = 1.0) -> np.ndarray:
    """fp64 samples at logical indices ``idx`` (any integer array)."""
    if dist == "zeros":
        return np.zeros(idx.shape, dtype=np.float64)
    x0, x1 = _raw(seed, tensor_id, idx)
    h0 = (x0 >> np.uint64(11)).astype(np.float64)
    if dist == "uniform":            # [-1, 1)
        return 2.0 * (h0 * 2.0 ** -53) - 1.0
    if dist == "normal":             # N(0, scale^2)
        u0 = (h0 + 1.0) * 2.0 ** -53
        u1 = (x1 >> np.uint64(11)).astype(np.float64) * 2.0 ** -53
        return scale * np.sqrt(-2.0 * np.log(u0)) * np.cos(2.0 * np.pi * u1)
    if dist == "smallint":           # integers in [-4, 4]
        return np.floor(h0 * 2.0 ** -53 * 9.0) - 4.0
    raise ValueError(f"unknown distribution {dist!r}")


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    w = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (w >> np.uint32(16)) & np.uint32(1)
    return ((w + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def tensor(seed: int, tensor_id: int, shape, dist: str, scale: float = 1.0, dtype: str = "bf16",
           colmajor_last2: bool = False) -> np.ndarray:
    """A whole tensor of logical ``shape``.

    ``dtype``: "bf16" (uint16 bits) or "f32".  With ``colmajor_last2`` the last two logical
    dimensions are stored transposed (the returned array has them swapped) while every element
    keeps the value of its LOGICAL row-major index.
    """
    shape = tuple(int(s) for s in shape)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == "bf16" else np.float32)

    def fill(lo):
        hi = min(n, lo + _CHUNK)
        v = values_f64(seed, tensor_id, np.arange(lo, hi, dtype=np.uint64), dist, scale)
        out[lo:hi] = f32_to_bf16_bits(v.astype(np.float32)) if dtype == "bf16" else v.astype(np.float32)

    starts = range(0, n, _CHUNK)
    if len(starts) > 1:       # chunks are independent (index-pure), numpy releases the GIL
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
            list(pool.map(fill, starts))
    else:
        for lo in starts:
            fill(lo)
    out = out.reshape(shape)
    if colmajor_last2:
        out = np.ascontiguousarray(np.swapaxes(out, -1, -2))
    return out
