"""Builds the CUDA library (sm_100a only) next to this file:  python paper_1811_02084_b200/build.py

Run it by path (not with -m): importing the package loads the library, which may not exist yet."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmtf_b200.so")
# Optional second library for single-GPU runs: the same sources plus csrc/tma_multicast.cuh (operand
# loads that write into several CTAs of a cluster).  Both that header and this library are left out
# of anything that runs on two or more GPUs; the package then uses LIB.
LIB_MC = os.path.join(HERE, "libmtf_b200_mc.so")
MC_HEADER = os.path.join(CSRC, "tma_multicast.cuh")
SOURCES = ["planner.cpp", "api.cpp", "blocks.cpp", "einsum_simt.cu", "gemm_tcgen05.cu", "rowwise.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "mtf.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def stale() -> bool:
    return _stale(LIB) or (os.path.exists(MC_HEADER) and _stale(LIB_MC))


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every source with nvcc for sm_100a into libmtf_b200.so.  Returns the library path."""
    if not force and not stale():
        return LIB
    srcs = [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    targets = [(LIB, [])]
    if os.path.exists(MC_HEADER):
        targets.append((LIB_MC, ["-DMTF_TMA_MULTICAST=1"]))
    for lib, extra in targets:
        if not force and not _stale(lib):
            continue
        tmp = lib + f".tmp{os.getpid()}"
        cmd = [_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + srcs
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or proc.returncode != 0:
            sys.stderr.write(proc.stdout + proc.stderr)
        if proc.returncode != 0:
            raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}:\n" + proc.stderr[-4000:])
        os.replace(tmp, lib)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
