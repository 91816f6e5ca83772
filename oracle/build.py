"""Compile the C oracle into oracle/libmodse_oracle.so (gcc, OpenMP).

Test infrastructure only.  Run as ``python -m oracle.build`` or call
``build()``; the shared object is rebuilt when the C source is newer.
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "modse_oracle.c")
HDR = os.path.join(HERE, "modse_oracle.h")
LIB = os.path.join(HERE, "libmodse_oracle.so")


def build(force: bool = False) -> str:
    newest = max(os.path.getmtime(SRC), os.path.getmtime(HDR))
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest:
        return LIB
    cmd = ["gcc", "-std=c99", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall",
           "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
