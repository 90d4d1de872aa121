"""Compile the oracle's C++ translation unit into oracle/liboracle.so (g++, OpenMP over rows)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "hqref.cpp")
LIB = os.path.join(HERE, "liboracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


def check_no_float_codegen() -> None:
    """Compile-only pass that forbids every floating-point / vector register (x86 GCC): the integer
    pipeline must build with general registers alone (the paper's no-floating-point claim)."""
    cmd = ["g++", "-std=c++17", "-O1", "-mgeneral-regs-only", "-fsyntax-only", "-c", SRC]
    subprocess.run(cmd, check=True)


if __name__ == "__main__":
    print(build(force=True))
