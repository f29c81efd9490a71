"""Compile the CPU oracle (test infrastructure) into oracle/libq4d_oracle.so with gcc.

Plain x86-64 code generation (no -march=native): the shared object may be built
on one machine and loaded on another.  Floating-point contraction is off so the
fp64 arithmetic is exactly what the source spells out.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "q4d_oracle.c")
LIB = os.path.join(HERE, "libq4d_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["gcc", "-std=c11", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
           "-shared", "-Wall", "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
