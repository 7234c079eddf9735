"""Compile the native parts in-tree: the CUDA library (nvcc, sm_100a) and the input generator (gcc)."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_ROOT = os.path.dirname(_HERE)
LIB_MDI = os.path.join(_HERE, "libmdi.so")
LIB_INPUTS = os.path.join(_HERE, "libmdi_inputs.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _stale(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build_inputs(force: bool = False) -> str:
    src = os.path.join(_CSRC, "synth_inputs.c")
    if force or _stale(LIB_INPUTS, [src]):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", LIB_INPUTS, src, "-lm"])
    return LIB_INPUTS


def build_mdi(force: bool = False, verbose: bool = False) -> str:
    cu = sorted(glob.glob(os.path.join(_CSRC, "*.cu")))
    if not cu:
        raise RuntimeError("no CUDA sources under csrc/")
    deps = cu + glob.glob(os.path.join(_CSRC, "*.cuh")) + glob.glob(os.path.join(_ROOT, "include", "*.h"))
    if force or _stale(LIB_MDI, deps):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-I", os.path.join(_ROOT, "include"), "-o", LIB_MDI] + cu
        subprocess.check_call(cmd)
    return LIB_MDI


def build_all(force: bool = False) -> None:
    build_inputs(force)
    build_mdi(force)


if __name__ == "__main__":
    import sys
    build_inputs("--force" in sys.argv)
    build_mdi("--force" in sys.argv, verbose="-v" in sys.argv)
