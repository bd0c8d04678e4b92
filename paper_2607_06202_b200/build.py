"""Builds the CUDA library in-tree: ``python -m paper_2607_06202_b200.build``."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libubep.so")
SOURCES = ["ubep_kernels.cu", "ubep_host.cu", "ubep_static.cu", "ubep_mapper.cu", "ubep_sync.cu", "ubep_sharded.cu"]
DEPENDS = SOURCES + ["ubep_common.cuh", "ubep_layout.cuh", "ubep_quant.cuh", "ubep_kernels.h", "ubep_sync.h", "ubep_sharded.h", "../../include/ubep.h"]


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(os.path.join(CSRC, d)) <= t for d in DEPENDS)


def build(force: bool = False, verbose: bool = False) -> str:
    """nvcc for sm_100a only; the library is a plain shared object with a C ABI."""
    if not force and up_to_date():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-o", LIB]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
