"""Compile the CPU oracle (oracle/tsq_ref.cpp) into oracle/libtsq_ref.so.

Test infrastructure: building the checker is not using it.  The flags pin the
arithmetic the oracle is defined in: IEEE binary32, no FMA contraction, no
fast-math, one thread.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "tsq_ref.cpp")
LIB = os.path.join(HERE, "libtsq_ref.so")

FLAGS = [
    "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fno-unsafe-math-optimizations",
    "-Wall", "-Wextra", "-shared", "-fPIC",
]


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its source; return its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = ["g++", *FLAGS, SRC, "-o", tmp]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("oracle build failed:\n%s\n%s" % (" ".join(cmd), res.stderr))
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
