"""Builds the CUDA library (sm_100a only) next to this file:  python paper_1811_02084_b200/build.py

Run it by path (not with -m): importing the package loads the library, which may not exist yet.

Every source is compiled to an object of its own (in parallel, cached under csrc/build/ by the
modification times of the sources) and the objects are linked into libmtf_b200.so."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libmtf_b200.so")
# Optional second library, for single-GPU runs that ask for it: the same objects except that the
# contraction kernel is compiled with csrc/tma_multicast.cuh force-included (operand loads that write
# into several CTAs of a cluster; the tensor maps they use cover this GPU's memory alone).  That
# header and this library are left out of anything that runs on two or more GPUs, no other source
# names what the header contains, and the package loads LIB unless told otherwise.
LIB_MC = os.path.join(HERE, "libmtf_b200_mc.so")
MC_HEADER = os.path.join(CSRC, "tma_multicast.cuh")
MC_SOURCE = "gemm_tcgen05.cu"
SOURCES = ["planner.cpp", "api.cpp", "blocks.cpp", "ranks.cpp", "chooser.cpp", "ops.cpp", "einsum_simt.cu", "gemm_tcgen05.cu", "rowwise.cu",
           "relayout.cu", "vocab.cu", "update.cu", "attention_fused.cu", "attention_bwd_fused.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh")) and f != os.path.basename(MC_HEADER)]
    return hs + [os.path.join(HERE, "..", "include", "mtf.h")]


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _obj(src: str, variant: str) -> str:
    return os.path.join(OBJ_DIR, f"{os.path.splitext(src)[0]}{variant}.o")


def _obj_stale(src: str, variant: str) -> bool:
    o = _obj(src, variant)
    if not os.path.exists(o):
        return True
    t = os.path.getmtime(o)
    deps = [os.path.join(CSRC, src)] + _headers() + ([MC_HEADER] if variant else [])
    return any(os.path.getmtime(d) > t for d in deps)


def _targets():
    """(library, [(source, variant)]) for every library to build."""
    srcs = _sources()
    out = [(LIB, [(s, "") for s in srcs])]
    if os.path.exists(MC_HEADER):
        out.append((LIB_MC, [(s, ".mc" if s == MC_SOURCE else "") for s in srcs]))
    return out


def _lib_stale(lib: str, objs) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(_obj_stale(s, v) or os.path.getmtime(_obj(s, v)) > t for s, v in objs)


def stale() -> bool:
    return any(_lib_stale(lib, objs) for lib, objs in _targets())


def _compile(src: str, variant: str, verbose: bool):
    extra = ["-include", MC_HEADER] if variant else []
    tmp = _obj(src, variant) + f".tmp{os.getpid()}"
    cmd = [_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", tmp, os.path.join(CSRC, src)]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode == 0:
        os.replace(tmp, _obj(src, variant))
    return src + variant, proc


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every source with nvcc for sm_100a and link libmtf_b200.so.  Returns the library path."""
    if not force and not stale():
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    todo = []
    for _lib, objs in _targets():
        for s, v in objs:
            if (force or _obj_stale(s, v)) and (s, v) not in todo:
                todo.append((s, v))
    with ThreadPoolExecutor(max_workers=max(1, min(len(todo), os.cpu_count() or 4))) as pool:
        results = list(pool.map(lambda sv: _compile(sv[0], sv[1], verbose), todo))
    for name, proc in results:
        if verbose or proc.returncode != 0:
            sys.stderr.write(f"---- {name}\n" + proc.stdout + proc.stderr)
        if proc.returncode != 0:
            raise RuntimeError(f"nvcc failed compiling {name}:\n" + proc.stderr[-4000:])
    for lib, objs in _targets():
        tmp = lib + f".tmp{os.getpid()}"
        cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + [_obj(s, v) for s, v in objs]
        proc = subprocess.run(cmd, capture_output=True, text=True)
        if proc.returncode != 0:
            raise RuntimeError(f"nvcc failed linking {os.path.basename(lib)}:\n" + proc.stderr[-4000:])
        os.replace(tmp, lib)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
