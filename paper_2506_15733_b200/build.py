"""Builds the C-ABI shared library from ``csrc/`` with nvcc for sm_100a, in-tree."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libspecs_b200.so")
LIB_PATH_DEBUG = os.path.join(PKG_DIR, "libspecs_b200_debug.so")   # the checked build (-DSPECS_DEBUG)
SOURCES = ["api.cu", "planner.cu", "score_tcgen05.cu", "score_simt.cu", "select_kernels.cu", "score_noalloc.cu", "controller.cpp"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found (set NVCC or put it on PATH)")


def needs_build(debug: bool = False) -> bool:
    lib = LIB_PATH_DEBUG if debug else LIB_PATH
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "specs.h")]
    return any(os.path.getmtime(p) > built for p in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every CUDA source for sm_100a into one shared library; returns its path.
    ``debug`` builds the checked library instead: index checks inside the kernels and the plain CUDA-core
    scoring engine (see specs_debug_build in specs.h)."""
    lib = LIB_PATH_DEBUG if debug else LIB_PATH
    if not force and not needs_build(debug):
        return lib
    cmd = [_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + (["-DSPECS_DEBUG"] if debug else []) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr, file=sys.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
