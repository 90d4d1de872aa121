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


def check_no_float_codegen(src: str = SRC) -> None:
    """Compile `src` to object code (discarded) with every floating-point / vector register forbidden
    (x86 GCC, -mgeneral-regs-only): the integer pipeline must build with general registers alone (the
    paper's no-floating-point claim, Section 1 and Appendix H).  GCC raises this error while generating
    code, so the pass has to compile for real: a syntax-only run accepts a `double`.
    Raises subprocess.CalledProcessError when the source needs a floating-point register."""
    cmd = ["g++", "-std=c++17", "-O1", "-mgeneral-regs-only", "-c", src, "-o", os.devnull]
    subprocess.run(cmd, check=True, stderr=subprocess.DEVNULL)


if __name__ == "__main__":
    print(build(force=True))
