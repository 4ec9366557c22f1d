"""Compile the float64 CPU oracle (oracle/kopref.c) into oracle/libkopref.so with gcc.

Test infrastructure: nothing in the product package imports this module.
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "kopref.c")
LIB = os.path.join(HERE, "libkopref.so")

# -ffp-contract=off: no fused multiply-add, so every operation rounds as written.
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
          "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Build the shared library if it is missing or older than its source; return its path."""
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    subprocess.run(["gcc", *CFLAGS, SRC, "-o", tmp, "-lm"], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
