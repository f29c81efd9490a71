"""Compile the CUDA sources of the decode-step library for sm_100a into
paper_2601_19139_b200/libq4decode.so (in-tree, next to this file)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libq4decode.so")
SOURCES = ["api.cu", "q4_gemm.cu", "q4_umma.cu", "attention.cu", "elementwise.cu", "moe.cu", "sampling.cu", "no_alloc.cu", "fused_step.cu", "cache.cpp"]


def _newest_source_mtime():
    times = [os.path.getmtime(os.path.join(CSRC, f)) for f in os.listdir(CSRC)]
    times.append(os.path.getmtime(os.path.join(HERE, "..", "include", "q4decode.h")))
    return max(times)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC", "-shared", "--threads", "4"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
