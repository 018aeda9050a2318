"""Builds libbitcos.so (CUDA kernels for sm_100a + host packers) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbitcos.so")
SOURCES = [os.path.join(CSRC, "gemv.cu"), os.path.join(CSRC, "probe.cu"), os.path.join(CSRC, "pack_device.cu"),
           os.path.join(CSRC, "pack.cpp")]
HEADERS = [os.path.join(ROOT, "include", "bitcos.h"), os.path.join(CSRC, "decode.cuh")]


def nvcc_command(extra=()):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
            "-I" + os.path.join(ROOT, "include"), "-Xcompiler", "-fPIC,-fopenmp,-O2", "-shared",
            "-o", LIB, *SOURCES, "-lgomp", *extra]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        cmd = nvcc_command(("-Xptxas", "-v") if verbose else ())
        subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
