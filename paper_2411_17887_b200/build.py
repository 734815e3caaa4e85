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


PROFILE_LIB = os.path.join(HERE, "libtcu_scan_profile.so")   # the debug build with per-role wait counters


def nvcc_command(out: str, verbose: bool = False, profile: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-o", out] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    if profile:
        cmd[1:1] = ["-DTCU_PROFILE"]
    return cmd


def build_profile(force: bool = False) -> str:
    """The same library compiled with -DTCU_PROFILE (the debug section of the kernel file: cycle counters of where
    each role waits).  Only ``bench.py --wait-counters`` loads it; the product never does."""
    if not force and os.path.exists(PROFILE_LIB) and all(os.path.getmtime(PROFILE_LIB) >= os.path.getmtime(d) for d in DEPENDS):
        return PROFILE_LIB
    tmp = PROFILE_LIB + f".tmp{os.getpid()}"
    subprocess.run(nvcc_command(tmp, profile=True), check=True)
    os.replace(tmp, PROFILE_LIB)
    return PROFILE_LIB


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile for sm_100a if the library is missing or older than its sources; return its path."""
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in DEPENDS):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run(nvcc_command(tmp, verbose), check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    if "--profile" in sys.argv:
        print(build_profile(force=True))
    else:
        print(build(force=True, verbose=True))
