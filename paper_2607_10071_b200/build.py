"""Build the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
SOURCES = [os.path.join(_HERE, "csrc", "flashbev.cu")]
HEADERS = [os.path.join(ROOT, "include", "flashbev.h"), os.path.join(_HERE, "csrc", "vt_tiled.cuh")]
LIB = os.path.join(_HERE, "libflashbev.so")

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include")]


LIB_DEBUG_BOUNDS = os.path.join(_HERE, "libflashbev_debug_bounds.so")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(s) > t for s in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile csrc/*.cu into libflashbev.so next to this file; returns its path.

    ``debug_bounds``: build libflashbev_debug_bounds.so instead, with -DFLASHBEV_DEBUG_BOUNDS: every index the
    tiled kernel computes is range-checked, violations are counted into the caller's ``debug_error_word`` and
    the access is redirected to a safe slot (the stand-in for a memory checker on machines where none may run)."""
    lib = LIB_DEBUG_BOUNDS if debug_bounds else LIB
    if force or needs_build(lib):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = ([nvcc] + NVCC_FLAGS + (["-DFLASHBEV_DEBUG_BOUNDS"] if debug_bounds else []) +
               (["-Xptxas", "-v"] if verbose else []) + SOURCES + ["-o", lib])
        subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
