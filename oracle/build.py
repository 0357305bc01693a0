"""Compile the float64 CPU oracle (plain C, gcc) into oracle/librapid_oracle.so.

Test infrastructure only: nothing in the CUDA library or its Python binding imports this.
"""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "rapid_oracle.c")
LIB = os.path.join(_HERE, "librapid_oracle.so")


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its source; return its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = [
        "gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
        "-o", LIB, SRC, "-lm",
    ]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
