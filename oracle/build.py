"""Compile the C oracle into ``oracle/liboracle.so`` with gcc.

Test infrastructure: the product library neither needs nor loads this file.
Run as ``python -m oracle.build`` or call :func:`build`.
"""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "attn_oracle.c")
LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its source."""
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
           "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
