"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libabs_b200.so")
SOURCES = [os.path.join(CSRC, "abs_b200.cu"), os.path.join(CSRC, "abs_gemm.cu")]
HEADERS = [os.path.join(CSRC, "abs_device.cuh"), os.path.join(CSRC, "abs_fast4.cuh"), os.path.join(CSRC, "abs_opt4.cuh"), os.path.join(CSRC, "abs_fastx.cuh"), os.path.join(CSRC, "abs_trans4.cuh"), os.path.join(CSRC, "abs_generic.cuh"), os.path.join(os.path.dirname(_HERE), "include", "abs_b200.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    # bit-exactness: no implicit multiply-add contraction, IEEE division / sqrt, subnormals kept
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "--shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-cudart", "static", "-Xlinker", "-Bsymbolic",
]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libabs_b200.so if it is missing or older than its sources. Returns its path."""
    if not force and not needs_build():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
