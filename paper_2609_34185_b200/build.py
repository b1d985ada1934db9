"""Builds the C-ABI library (host encoder + sm_100a decode kernels) in-tree with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libentropack_b200.so")
SOURCES = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")) + glob.glob(os.path.join(HERE, "csrc", "*.cpp")))
HEADERS = sorted(glob.glob(os.path.join(HERE, "csrc", "*.hpp")) + glob.glob(os.path.join(ROOT, "include", "*.h")))


def nvcc_command(out: str = LIB, verbose: bool = False) -> list[str]:
    nvcc = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-ffp-contract=off,-pthread", "-shared", "-I", os.path.join(ROOT, "include"),
           "-o", out]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    return cmd + SOURCES


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        subprocess.run(nvcc_command(verbose=verbose), check=True, cwd=ROOT)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
