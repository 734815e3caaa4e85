"""Compile the plain-C result oracle into a shared object next to its source.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Usage::

    python -m oracle.build
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "scan_oracle.c")
LIB = os.path.join(HERE, "libscan_oracle.so")


def build(force: bool = False) -> str:
    """Build ``libscan_oracle.so`` with gcc if it is missing or stale; return its path."""
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    # -O1 and no fast-math: the loop must stay a sequential left-to-right sum.
    cmd = ["gcc", "-O1", "-fno-fast-math", "-shared", "-fPIC", "-o", tmp, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
