"""Seeded synthetic input generator shared by the tests, the bench and the oracle checks.

This module holds no arithmetic of the method (no einsum, no slicing, no layout logic).  It only
produces reproducible arrays of random numbers and rounds them to a storage type, so that the CPU
oracle and the CUDA path can be handed byte-identical inputs.

Generator: counter based.  Element ``i`` of the stream ``(seed, name)`` is a pure function of
``(seed, name, i)``:

    key  = splitmix64(seed XOR fnv1a64(name))
    u1   = (splitmix64(key + 2i)     >> 11 + 1) / 2**53      in (0, 1]
    u2   = (splitmix64(key + 2i + 1) >> 11)     / 2**53      in [0, 1)
    z_i  = sqrt(-2 ln u1) * cos(2 pi u2)                     standard normal (Box-Muller), fp64

so results do not depend on numpy's or torch's random generators or on the chunking used here.
Values are then scaled in fp64 and rounded once to the storage type: ``f32`` (IEEE round to nearest
even) or ``bf16`` (fp64 -> fp32 -> round-to-nearest-even on the top 16 bits).
"""
from __future__ import annotations

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_CHUNK = 1 << 22


def fnv1a64(name: str) -> int:
    h = 0xCBF29CE484222325
    for b in name.encode("utf-8"):
        h ^= b
        h = (h * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _splitmix64_scalar(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return z ^ (z >> 31)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 finaliser on uint64 (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = x + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def stream_key(seed: int, name: str) -> int:
    return _splitmix64_scalar((int(seed) ^ fnv1a64(name)) & 0xFFFFFFFFFFFFFFFF)


def normal_f64(seed: int, name: str, count: int, start: int = 0) -> np.ndarray:
    """Elements ``start .. start+count-1`` of the standard-normal stream ``(seed, name)``, fp64."""
    key = np.uint64(stream_key(seed, name))
    out = np.empty(count, dtype=np.float64)
    two53 = float(1 << 53)
    for c0 in range(0, count, _CHUNK):
        n = min(_CHUNK, count - c0)
        i = np.arange(start + c0, start + c0 + n, dtype=np.uint64)
        with np.errstate(over="ignore"):
            a = _splitmix64(key + np.uint64(2) * i)
            b = _splitmix64(key + np.uint64(2) * i + np.uint64(1))
        u1 = ((a >> np.uint64(11)).astype(np.float64) + 1.0) / two53
        u2 = (b >> np.uint64(11)).astype(np.float64) / two53
        out[c0:c0 + n] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp64/fp32 array -> uint16 bf16 bit patterns (via fp32, round to nearest even)."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


class Stored:
    """A generated tensor in its storage type.

    ``bits``  : the bytes the device gets (np.float32 array, or np.uint16 array of bf16 patterns)
    ``f64``   : exactly the same values widened to fp64 (what a CPU checker reads)
    ``dtype`` : "f32" or "bf16"
    """

    __slots__ = ("bits", "f64", "dtype", "shape")

    def __init__(self, bits: np.ndarray, f64: np.ndarray, dtype: str):
        self.bits = bits
        self.f64 = f64
        self.dtype = dtype
        self.shape = tuple(bits.shape)


def store(values_f64: np.ndarray, dtype: str) -> Stored:
    """Round an fp64 array once to ``dtype`` and return both representations."""
    v = np.ascontiguousarray(values_f64, dtype=np.float64)
    if dtype == "f32":
        b = v.astype(np.float32)
        return Stored(b, b.astype(np.float64), "f32")
    if dtype == "bf16":
        b = round_to_bf16_bits(v)
        return Stored(b, bf16_bits_to_f64(b).reshape(v.shape), "bf16")
    raise ValueError(f"unknown storage dtype {dtype!r}")


def normal(seed: int, name: str, shape, dtype: str, scale: float = 1.0, shift: float = 0.0) -> Stored:
    """``shift + scale * N(0,1)`` of the given shape, rounded to ``dtype``."""
    shape = tuple(int(s) for s in shape)
    n = int(np.prod(shape, dtype=np.int64)) if shape else 1
    z = normal_f64(seed, name, n).reshape(shape)
    return store(shift + scale * z, dtype)


def small_integers(seed: int, name: str, shape, lo: int = -4, hi: int = 4) -> np.ndarray:
    """Integer-valued fp64 array with entries in [lo, hi] (exact sums in any order)."""
    shape = tuple(int(s) for s in shape)
    n = int(np.prod(shape, dtype=np.int64)) if shape else 1
    key = np.uint64(stream_key(seed, name))
    with np.errstate(over="ignore"):
        r = _splitmix64(key + np.arange(n, dtype=np.uint64))
    span = np.uint64(hi - lo + 1)
    return ((r % span).astype(np.int64) + lo).astype(np.float64).reshape(shape)


def sample_indices(seed: int, name: str, extent: int, count: int, must_include=()) -> np.ndarray:
    """Sorted unique indices in [0, extent): ``must_include`` plus seeded picks, at most ``count`` new."""
    key = np.uint64(stream_key(seed, name))
    with np.errstate(over="ignore"):
        r = _splitmix64(key + np.arange(count, dtype=np.uint64))
    picks = (r % np.uint64(extent)).astype(np.int64)
    inc = np.asarray([i for i in must_include if 0 <= i < extent], dtype=np.int64)
    return np.unique(np.concatenate([inc, picks]))
