"""A second build of the oracle's source in which the projections accumulate in fp32 instead of fp64.

It is NOT the oracle: it exists to measure how far a correct implementation that differs from the definition only in
accumulation precision drifts once bf16 rounding decisions start to differ (every GPU kernel accumulates in fp32).
The drift test compares the GPU's distance from the oracle with this variant's distance from the oracle.  The shared
object is written under tests/_build/ and loaded only here.
"""
import contextlib
import ctypes as C
import os
import subprocess

from oracle import q4d_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "..", "oracle", "q4d_oracle.c")
OUT_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(OUT_DIR, "libq4d_oracle_fp32probe.so")

_PROBE = None


def _lib():
    global _PROBE
    if _PROBE is None:
        os.makedirs(OUT_DIR, exist_ok=True)
        if not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
            subprocess.run(["gcc", "-std=c11", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
                            "-DORC_SENSITIVITY_PROBE_FP32", "-o", LIB, SRC, "-lm"], check=True)
        _PROBE = orc._declare(C.CDLL(LIB))
    return _PROBE


@contextlib.contextmanager
def fp32_accumulation():
    """While active, the oracle's Python wrapper calls the fp32-accumulating variant."""
    orc.lib()
    saved, orc._LIB = orc._LIB, _lib()
    try:
        yield
    finally:
        orc._LIB = saved
