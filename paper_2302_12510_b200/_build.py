"""Builds libdybit.so in-tree with nvcc for sm_100a (no JIT cache, no fallback)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libdybit.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libdybit_debug.so")     # the same sources with -DDYBIT_DEBUG_BOUNDS (range checks)
_SOURCES = [os.path.join(_PKG, "csrc", "dybit_lib.cu")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-std=c++17", "-O3", "-lineinfo",
    "-shared", "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libdybit.so cannot be built")
    return exe


def _deps():
    return (glob.glob(os.path.join(_PKG, "csrc", "*")) +
            glob.glob(os.path.join(_ROOT, "include", "*.h")))


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(p) > t for p in _deps())


def build_library(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile the CUDA sources into paper_2302_12510_b200/libdybit.so (or, with debug_bounds, into
    libdybit_debug.so: the build whose global stores are range-checked, see DYBIT_CHECK in csrc/dybit_common.cuh)."""
    out = DEBUG_LIB_PATH if debug_bounds else LIB_PATH
    if not force and not is_stale(out):
        return out
    tmp = out + ".tmp%d" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + (["-DDYBIT_DEBUG_BOUNDS"] if debug_bounds else []) + (["-Xptxas", "-v"] if verbose else []) + [
        "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_PKG, "csrc"),
        "-o", tmp] + _SOURCES
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout + proc.stderr)
    if verbose:
        print(proc.stderr)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    import sys
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
