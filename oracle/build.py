"""Compile the oracle's C source into ``oracle/liboracle.so`` with gcc.

Plain ``-O2`` with OpenMP over rows and no fast-math: the oracle is a checker, it is
never tuned.  Building the checker is not using it; the product never loads it.
"""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC_PATH = os.path.join(_HERE, "ak_oracle.c")
LIB_PATH = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB_PATH)
            and os.path.getmtime(LIB_PATH) >= os.path.getmtime(SRC_PATH)):
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-fopenmp",
           "-fno-fast-math", "-ffp-contract=off",
           "-Wall", "-Wextra", "-o", tmp, SRC_PATH, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB_PATH)  # atomic: concurrent test workers never see a partial file
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True))
