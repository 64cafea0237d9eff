"""Builds libkvt.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libkvt.so")
SOURCES = ["kvt_engine.cu"]
DEPS = ["kvt_kernels.cuh", os.path.join("..", "..", "include", "kvt.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC"]
DEFINES: list = []


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_HERE, "..", "include", "kvt.h")]
    return any(os.path.getmtime(f) > t for f in files)


DEBUG_LIB = os.path.join(_HERE, "libkvt_debug.so")


def build_debug_lib(force: bool = False) -> str:
    """The checked build of the same sources (-DKVT_DEBUG): index / invariant checks in the kernels that set the
    device error word, and every launch in another shape (64-thread blocks, a handful of mover CTAs, no CUDA
    graph). Load it with KVT_LIB=<path>. Used by the tests; the product is libkvt.so."""
    return build_lib(force, lib=DEBUG_LIB, defines=["-DKVT_DEBUG"])


def build_lib(force: bool = False, verbose: bool = False, lib: str = LIB, defines=None) -> str:
    """Compiles libkvt.so if it is missing or older than its sources. Safe when several processes call it at once
    (one rank per GPU): an exclusive file lock serialises them, the compiler writes to a temporary file and the
    result is moved into place in one step, so nobody ever loads a half-written library."""
    if not (force or _stale(lib)):
        return lib
    import fcntl
    with open(lib + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if force or _stale(lib):         # somebody else may have built it while we waited
                nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
                tmp = f"{lib}.{os.getpid()}.tmp"
                cmd = [nvcc] + NVCC_FLAGS + DEFINES + list(defines or []) + (["-Xptxas", "-v"] if verbose else []) + \
                      ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
                try:
                    subprocess.check_call(cmd)
                    os.replace(tmp, lib)
                finally:
                    if os.path.exists(tmp):
                        os.remove(tmp)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return lib


TRACE_LIB = os.path.join(_HERE, "libkvt_trace.so")


def build_trace_lib(force: bool = False) -> str:
    """Development build with per-kernel event timing (-DKVT_TRACE): with KVT_TRACE=1 in the environment the LOOKUP
    and selection calls print the time between their launches to stderr; KVT_NO_OVERLAP=1 launches the LOOKUP kernels
    without the tail overlap, KVT_NO_GRAPH=1 the selection without its CUDA graph. Load it with KVT_LIB=<path>."""
    return build_lib(force, lib=TRACE_LIB, defines=["-DKVT_TRACE"])


if __name__ == "__main__":
    import sys
    if "--trace" in sys.argv:
        print(build_trace_lib(force=True))
    else:
        print(build_lib(force=True, verbose="-v" in sys.argv))
