"""TEST INFRASTRUCTURE.  Storage rounding used when the oracle models WHERE the method keeps a tensor
in a narrow type between two einsums.

The precision contract of the GPU path is "bf16 storage, fp32 accumulation, round to nearest even":
each einsum reads bf16 tensors and its result is rounded once when it is stored.  The oracle's
arithmetic stays fp64; `store` is the single rounding of a stored intermediate (the hidden
activations h and the gradient dhp of the feed-forward block; q, k, v, the attention weights and o
of the attention block).  With ``dtype=None`` nothing is rounded and the blocks are exact mathematics.
"""
from __future__ import annotations

import numpy as np


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp64 -> nearest bf16 (ties to even), returned as fp64.  Goes through fp32 first, as a
    conversion of an fp32 accumulator does."""
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    out = r.astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(np.isfinite(f), out, f.astype(np.float64))


def round_to_f32(a: np.ndarray) -> np.ndarray:
    return np.asarray(a, dtype=np.float64).astype(np.float32).astype(np.float64)


def make_store(ops, dtype):
    """Returns a function tensor -> tensor that rounds to the storage dtype through ``ops.unary``."""
    if dtype is None:
        return lambda t: t
    fn = {"bf16": round_to_bf16, "f32": round_to_f32}[dtype]
    return lambda t: ops.unary(t, fn)
