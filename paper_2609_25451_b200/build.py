"""Builds the C-ABI shared library (``libgms.so``) in-tree with nvcc for sm_100a.

    python -m paper_2609_25451_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU; the library links the static CUDA runtime and
has no Python or torch dependency.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libgms.so")
SOURCES = ["gms_api.cu", "gms_stream_kernels.cu", "gms_verify_kernels.cu", "gms_build_kernels.cu", "gms_noalloc.cu", "gms_pipe.cu",
           "gms_service.cu"]
HEADERS = [os.path.join(CSRC, "gms_internal.h"), os.path.join(ROOT, "include", "gms.h")]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    cmd = [
        _nvcc(), "-std=c++17", "-O3", "-lineinfo",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "-Xcompiler", "-fPIC,-Wall,-Wextra", "-shared",
        "-I", os.path.join(ROOT, "include"),
        "-o", LIB,
    ] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
