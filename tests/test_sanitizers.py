"""The oracle (plain C) and the host side of the library (plan, permutation tables, validation, serialisation,
Gram post-processing) under AddressSanitizer and UndefinedBehaviorSanitizer: both are rebuilt with the
sanitizers, and the tests that need no GPU -- the oracle's pins and the host ABI checks -- run against those
builds in a child process with the sanitizer run-times preloaded.  A heap overrun, a use after free, a signed
overflow or a misaligned access in either fails the child.  Also checks that the NVTX build flag compiles."""
import os
import subprocess
import sys

import pytest

from paper_2505_11204_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _runtime(name):
    path = subprocess.run(["gcc", "-print-file-name=" + name], capture_output=True, text=True).stdout.strip()
    return path if os.path.isabs(path) and os.path.exists(path) else None


RUNNER = """
import os, sys
sys.path.insert(0, {root!r})
import oracle.randes_oracle as ro
ro._LIB = {oracle_lib!r}
from paper_2505_11204_b200 import randes, build
randes.LIB_PATH = {lib!r}
build.build_library = lambda *a, **k: randes.LIB_PATH
import pytest
rc = pytest.main(["-x", "-q", "-p", "no:cacheprovider", os.path.join({root!r}, "tests", "test_host_abi.py"),
                  os.path.join({root!r}, "tests", "test_oracle_pins.py"), "-k", "not missing_library"])
loaded = open("/proc/self/maps").read()
assert {lib!r} in loaded and {oracle_lib!r} in loaded and "libasan" in loaded, "the sanitized builds were not the ones loaded"
sys.exit(rc)
"""


def test_oracle_and_host_code_are_clean_under_asan_and_ubsan(tmp_path):
    asan, ubsan = _runtime("libasan.so"), _runtime("libubsan.so")
    if not asan or not ubsan:
        pytest.skip("gcc's sanitizer run-times are not installed")
    oracle_lib = str(tmp_path / "librandes_oracle_san.so")
    subprocess.run(["gcc", "-std=c11", "-O1", "-g", "-fno-omit-frame-pointer", "-fsanitize=address,undefined",
                    "-fno-sanitize-recover=undefined", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
                    "-o", oracle_lib, os.path.join(ROOT, "oracle", "randes_oracle.c"), "-lm"], check=True)
    lib = str(tmp_path / "librandes_san.so")
    subprocess.run(build.nvcc_command(lib, build.SANITIZER_FLAGS, opt="-O1"), check=True)
    env = dict(os.environ)
    env.update(LD_PRELOAD=asan + ":" + ubsan,
               ASAN_OPTIONS="detect_leaks=0:detect_odr_violation=0:verify_asan_link_order=0",
               UBSAN_OPTIONS="print_stacktrace=1:halt_on_error=1")
    r = subprocess.run([sys.executable, "-c", RUNNER.format(root=ROOT, oracle_lib=oracle_lib, lib=lib)], env=env,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-3000:])
    assert "runtime error" not in r.stderr and "AddressSanitizer" not in r.stderr, r.stderr[-3000:]


def test_nvtx_build_flag_compiles(tmp_path):
    """-DRANDES_NVTX (python -m paper_2505_11204_b200.build --nvtx) brackets every entry point with a named range;
    the host file that holds them must compile with the flag."""
    src = os.path.join(ROOT, "paper_2505_11204_b200", "csrc", "randes_api.cu")
    obj = str(tmp_path / "randes_api_nvtx.o")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc, "-O1", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC", "-DRANDES_NVTX",
                    "-c", src, "-o", obj], check=True)
    syms = subprocess.run(["nm", "-C", obj], capture_output=True, text=True).stdout
    assert "nvtxRangePushA" in syms or "nvtx" in syms.lower()
