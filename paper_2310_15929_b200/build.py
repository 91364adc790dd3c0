"""Builds libesparse.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libesparse.so")
HEADER = os.path.join(os.path.dirname(_PKG), "include", "esparse.h")
# Optional companion (single-GPU use only): its source and the built object are left out of multi-GPU runs.
MC_SOURCE = os.path.join(_CSRC, "spgemm_mcast.cu")
MC_LIB_PATH = os.path.join(_PKG, "libesparse_mc.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def _sources():
    return sorted(glob.glob(os.path.join(_CSRC, "*.cu")) + glob.glob(os.path.join(_CSRC, "*.cuh")) + [HEADER])


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(s) > t for s in _sources())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/esparse_lib.cu (one translation unit including the other .cu files) and, when its source is
    present, the optional companion library with the cluster-multicast form of the pair kernel."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    if force or is_stale():
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + [
            "-o", LIB_PATH, os.path.join(_CSRC, "esparse_lib.cu")]
        subprocess.run(cmd, check=True)
    if os.path.exists(MC_SOURCE) and (force or not os.path.exists(MC_LIB_PATH)
                                      or any(os.path.getmtime(s) > os.path.getmtime(MC_LIB_PATH) for s in _sources())):
        cmd = [nvcc] + NVCC_FLAGS + ["-Xcompiler", "-fvisibility=hidden"] + (["-Xptxas", "-v"] if verbose else []) + [
            "-o", MC_LIB_PATH, MC_SOURCE]
        subprocess.run(cmd, check=True)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
