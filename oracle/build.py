"""Compile the C oracle into oracle/libcmoe_oracle.so (gcc, OpenMP, no fast-math)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "cmoe_oracle.c")
LIB = os.path.join(HERE, "libcmoe_oracle.so")


def build(force: bool = False) -> str:
    deps = [SRC, os.path.join(HERE, "cmoe_oracle.h")]
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(p) for p in deps):
        return LIB
    # no -march=native: the object is built on one machine and may be loaded on another
    cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra",
           "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
