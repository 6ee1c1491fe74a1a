"""Builds libk2d.so (the sm_100a CUDA library behind include/k2d.h) in-tree with nvcc.

The arithmetic flags are part of the library's contract: no implicit multiply-add fusion, IEEE
division and square root, denormals kept, so that results are reproducible bit for bit.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(HERE, "csrc", "k2d_api.cu")
DEPS = [SRC, os.path.join(HERE, "csrc", "k2d_kernels.cuh"), os.path.join(ROOT, "include", "k2d.h")]
LIB = os.path.join(HERE, "libk2d.so")

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "--fmad=false", "--prec-div=true", "--prec-sqrt=true", "--ftz=false",
    "-Xcompiler", "-fPIC,-ffp-contract=off,-fno-fast-math", "-shared",
]


LIB_CHECKED = os.path.join(HERE, "libk2d_checked.so")
LIB_PHASES = os.path.join(HERE, "libk2d_phases.so")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False, checked: bool = False, phase_clocks: bool = False) -> str:
    """The library, or (checked=True) the build with index checks in the kernels (-DK2D_CHECKED), or (phase_clocks=True)
    the build whose step kernel adds up the cycles spent per phase of a step (-DK2D_PHASE_CLOCKS)."""
    if checked and phase_clocks:
        raise ValueError("one variant at a time")
    lib = LIB_CHECKED if checked else (LIB_PHASES if phase_clocks else LIB)
    if not force and not needs_build(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    defines = (["-DK2D_CHECKED"] if checked else []) + (["-DK2D_PHASE_CLOCKS"] if phase_clocks else [])
    cmd = [nvcc, *NVCC_FLAGS, *defines, "-I", os.path.join(ROOT, "include"), "-o", lib, SRC]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv, phase_clocks="--phase-clocks" in sys.argv))
