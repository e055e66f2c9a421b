"""TEST INFRASTRUCTURE.  Builds and loads the oracle's C loop nest (einsum_loops.c) with gcc."""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "einsum_loops.c")
_LIB = os.path.join(_HERE, "_einsum_loops.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile einsum_loops.c into a shared object next to it (a few hundred ms)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = ctypes.CDLL(_LIB)
            L.oracle_einsum_f64.restype = ctypes.c_int
            L.oracle_einsum_f64.argtypes = [
                ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p,
            ]
            _lib = L
        return _lib


def einsum_loops(sizes, in_strides, out_strides, n_out, inputs, out):
    """Call the C loop nest.  ``inputs``/``out`` are C-contiguous or strided fp64 numpy arrays; strides
    are in elements and given explicitly (0 = broadcast)."""
    n_in = len(inputs)
    nd = len(sizes)
    n_red = nd - n_out
    c_sizes = (ctypes.c_int64 * max(nd, 1))(*sizes)
    flat = [s for row in in_strides for s in row]
    c_in_strides = (ctypes.c_int64 * max(len(flat), 1))(*flat)
    c_out_strides = (ctypes.c_int64 * max(n_out, 1))(*out_strides)
    ptrs = (ctypes.c_void_p * n_in)(*[a.ctypes.data for a in inputs])
    for a in list(inputs) + [out]:
        assert a.dtype == np.float64
    rc = lib().oracle_einsum_f64(n_in, n_out, n_red, c_sizes, c_in_strides, c_out_strides, ptrs, out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"oracle_einsum_f64 rejected its arguments (code {rc})")
