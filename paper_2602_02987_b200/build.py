"""Builds libqsim.so (the C-ABI library of include/qsim.h) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libqsim.so")
SOURCES = [os.path.join(CSRC, "qsim_lib.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, "qsim_device.cuh"), os.path.join(CSRC, "qsim_lane.cuh"), os.path.join(CSRC, "qsim_ctmc.cuh"),
                     os.path.join(ROOT, "include", "qsim.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",                              # clocks are bit-exact: no fused multiply-add contraction
    "-Xcompiler", "-fPIC,-ffp-contract=off",
    "-shared",
]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in DEPENDS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if force or is_stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", LIB] + SOURCES
        subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
