"""Build the C-ABI library ``libfq.so`` (nvcc, sm_100a) and the generator's ``libfq_synth.so`` in-tree."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfq.so")
SOURCES = [os.path.join(CSRC, "fq_host.cpp"), os.path.join(CSRC, "fq_kernels.cu")]
HEADERS = [os.path.join(CSRC, "fq_internal.h"), os.path.join(CSRC, "fq_tc_kernel.cuh"), os.path.join(CSRC, "fq_mma_kernel.cuh"),
           os.path.join(CSRC, "fq_direct_kernel.cuh"), os.path.join(ROOT, "include", "fq.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-fopenmp,-ffp-contract=off,-fno-fast-math", "-shared",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build_lib(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + SOURCES + ["-lgomp"]
        subprocess.run(cmd, check=True)
    return LIB


def build_all(force: bool = False, verbose: bool = False) -> None:
    build_lib(force, verbose)
    from . import synth
    synth.build(force)


if __name__ == "__main__":
    sys.path.insert(0, ROOT)
    build_all(force="--force" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
