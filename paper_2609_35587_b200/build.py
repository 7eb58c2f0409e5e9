"""Build libks.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every .cu file is compiled to an object of its own (in parallel) under build/, then linked.
``build(debug=True)`` makes libks_debug.so instead: the same sources with KS_DEBUG_BOUNDS
defined, in which the kernels range-check the indices they form from data and record the
first violation in a word the host can read (``ks_debug_bounds_line``) instead of touching
memory out of range.
"""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libks.so")
LIB_DEBUG = os.path.join(_HERE, "libks_debug.so")
OBJ_DIR = os.path.join(_ROOT, "build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--extended-lambda", "-Xcompiler", "-fPIC"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) \
        + [os.path.join(_ROOT, "include", "ks.h")]


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not (force or stale(lib)):
        return lib
    tag = "debug" if debug else "release"
    os.makedirs(os.path.join(OBJ_DIR, tag), exist_ok=True)
    flags = NVCC_FLAGS + ["-I", os.path.join(_ROOT, "include"), "-I", CSRC]
    if debug:
        flags += ["-DKS_DEBUG_BOUNDS"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    newest_header = max(os.path.getmtime(h) for h in _headers())

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ_DIR, tag, os.path.basename(src)[:-3] + ".o")
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header):
            subprocess.run(["nvcc"] + flags + ["-c", "-o", obj, src], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    subprocess.run(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib] + objs, check=True)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
