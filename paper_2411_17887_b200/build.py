"""Build the C-ABI CUDA library in-tree (``libtcu_scan.so`` beside this file).

    python -m paper_2411_17887_b200.build
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libtcu_scan.so")
SOURCES = [os.path.join(HERE, "csrc", "tcu_scan.cu")]
DEPENDS = SOURCES + [os.path.join(HERE, "csrc", "tcu_scan_kernel.cuh"), os.path.join(ROOT, "include", "tcu_scan.h")]


def nvcc_command(out: str, verbose: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-o", out] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile for sm_100a if the library is missing or older than its sources; return its path."""
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in DEPENDS):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run(nvcc_command(tmp, verbose), check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
