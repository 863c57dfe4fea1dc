"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libcoral_lmhead.so")
LIB_CHECKED = os.path.join(PKG, "libcoral_lmhead_checked.so")   # same sources with -DCORAL_CHECK_BOUNDS
SOURCES = [os.path.join(CSRC, "coral_lmhead.cu")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def _newest_source_mtime() -> float:
    t = 0.0
    for d in (CSRC, os.path.join(ROOT, "include")):
        for f in os.listdir(d):
            t = max(t, os.path.getmtime(os.path.join(d, f)))
    return t


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """checked=True builds the range-checked variant: every index the kernels derive from the router's output
    is compared with the capacity of what it indexes (a violation sets CORAL_ERR_BOUNDS and skips the access).
    Load it by setting CORAL_LMHEAD_LIB to its path before the package is imported."""
    out = LIB_CHECKED if checked else LIB
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest_source_mtime():
        return out
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", out, *SOURCES]
    if checked:
        cmd.insert(1, "-DCORAL_CHECK_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return out


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
