"""Builds the CPU oracle (test infrastructure) into oracle/liboracle_ssdi8.so.

Strict IEEE binary32/binary64 arithmetic is part of the oracle's definition:
no contraction into fused multiply-adds, no fast-math, no -march flags (the
library is built on one machine and may run on another).
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ssdi8_oracle.cpp")
LIB = os.path.join(HERE, "liboracle_ssdi8.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-fPIC", "-shared", "-Wall", "-Wextra", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
