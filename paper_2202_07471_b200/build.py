"""Compile the CUDA library for sm_100a into paper_2202_07471_b200/libsquant.so (in-tree)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsquant.so")
LIB_DEBUG = os.path.join(HERE, "libsquant_debug.so")   # the checked build (-DSQUANT_DEBUG_BOUNDS), for tests on small cases
SOURCES = [os.path.join(CSRC, "squant.cu")]
DEPS = SOURCES + sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + [os.path.join(ROOT, "include", "squant.h")]

# -fmad=false: the solver's fp32 steps (division, rounding, difference) are written with
# explicit round-to-nearest intrinsics; no contraction is wanted anywhere else either.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-fmad=false", "--shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
              "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def nvcc_path() -> str:
    p = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(p):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return p


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and os.path.exists(lib) and all(
            os.path.getmtime(lib) >= os.path.getmtime(d) for d in DEPS):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [nvcc_path(), *NVCC_FLAGS, *(["-DSQUANT_DEBUG_BOUNDS"] if debug else []), "-o", tmp, *SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout)
        print(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, debug=True))
