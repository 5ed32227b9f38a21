"""Builds libfsoftmax.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfsoftmax.so")
LIB_DEBUG = os.path.join(HERE, "libfsoftmax_debug.so")      # the checked build: -DFS_DEBUG_BOUNDS
SOURCES = [os.path.join(CSRC, "fsoftmax.cu")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-cudart", "static", "-Xcompiler", "-fPIC", "-shared"]


def _inputs():
    files = list(SOURCES)
    for root, _, names in os.walk(CSRC):
        files += [os.path.join(root, n) for n in names if n.endswith((".cuh", ".h"))]
    files.append(os.path.join(os.path.dirname(HERE), "include", "fsoftmax.h"))
    return files


def nvcc_path() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libfsoftmax cannot be built")


def _command(lib: str, debug: bool, verbose: bool):
    cmd = [nvcc_path(), *NVCC_FLAGS, "-o", lib + ".tmp", *SOURCES]
    if debug:
        cmd.insert(1, "-DFS_DEBUG_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    return cmd


def _stale(lib: str) -> bool:
    return not os.path.exists(lib) or os.path.getmtime(lib) < max(os.path.getmtime(f) for f in _inputs())


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile if the shared object is missing or older than any source. Returns its path.
    debug=True builds the checked library (every global access range-checked) instead."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    subprocess.run(_command(lib, debug, verbose), check=True)
    os.replace(lib + ".tmp", lib)
    return lib


def build_all(force: bool = False):
    """Both builds, compiled side by side. Returns (normal, checked) paths."""
    jobs = [(lib, subprocess.Popen(_command(lib, dbg, False))) for lib, dbg in ((LIB, False), (LIB_DEBUG, True))
            if force or _stale(lib)]
    for lib, proc in jobs:
        if proc.wait() != 0:
            raise subprocess.CalledProcessError(proc.returncode, "nvcc")
        os.replace(lib + ".tmp", lib)
    return LIB, LIB_DEBUG


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
