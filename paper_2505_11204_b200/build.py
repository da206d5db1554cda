"""Compile the CUDA library for sm_100a into the package directory.

    python -m paper_2505_11204_b200.build [--force] [--verbose] [--nvtx] [--checked]

--nvtx brackets every computing entry point with an NVTX range (off by default).
--checked builds the kernels with their bounds predicates (slower; see randes_debug_violation).

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


def nvcc_command(out: str, extra_flags=(), opt: str = "-O3"):
    """The one nvcc invocation that builds the library into `out`."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return ([nvcc, opt, "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "--threads", "0",
             "-Xcompiler", "-fPIC", "-shared", "-o", out] + list(extra_flags) + [os.path.join(CSRC, s) for s in SOURCES])


# host code of the library under AddressSanitizer and UndefinedBehaviorSanitizer (device code is unaffected);
# load the result with the sanitizer run-times preloaded
SANITIZER_FLAGS = ["-Xcompiler", "-fsanitize=address,-fsanitize=undefined,-fno-sanitize-recover=undefined,-fno-omit-frame-pointer", "-g"]
# every computing entry point bracketed by an NVTX range named after it
NVTX_FLAGS = ["-DRANDES_NVTX", "-ldl"]
# the streaming kernels check the indices of every tile against the plan's bounds (randes_debug_violation)
CHECKED_FLAGS = ["-DRANDES_CHECKED"]


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), out: str = LIB) -> str:
    """Build the library (into the package directory unless `out` names another file)."""
    if out == LIB and not force and not _stale():
        return LIB
    tmp = out + ".%d.tmp" % os.getpid()
    flags = list(extra_flags) + (["-Xptxas", "-v"] if verbose else [])
    subprocess.run(nvcc_command(tmp, flags), check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    flags = (NVTX_FLAGS if "--nvtx" in sys.argv else []) + (CHECKED_FLAGS if "--checked" in sys.argv else [])
    print(build_library(force="--force" in sys.argv or bool(flags), verbose="--verbose" in sys.argv, extra_flags=flags))
