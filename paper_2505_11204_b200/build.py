"""Compile the CUDA library for sm_100a into the package directory.

    python -m paper_2505_11204_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  The shared object is kept in-tree (it is
not committed) so that it travels with the source tree to the machine that has
the GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librandes.so")
SOURCES = ["randes_api.cu", "randes_kernels.cu", "randes_group.cu", "randes_linear.cu", "randes_context.cu", "randes_batch.cu", "randes_diag.cu"]
HEADERS = [os.path.join(CSRC, "randes_internal.h"), os.path.join(CSRC, "randes_device.cuh"), os.path.join(os.path.dirname(HERE), "include", "randes.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += list(extra_flags)
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
