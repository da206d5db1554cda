"""The checked build of the library (-DRANDES_CHECKED): the streaming kernels compare the indices of every tile --
its layer, the layers and slots it reaches through the permutation tables, its rows -- with the plan's bounds before
they touch it, and keep the first failure in a device word.  Here that build is compiled and a cross-section of the
parity tests (ragged shapes, both storage types, groups, batches, random plans) runs against it in a child process:
the results must still equal the oracle's bit for bit, and the word must still be zero at the end."""
import os
import subprocess
import sys

import pytest

from paper_2505_11204_b200 import build, randes

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RUNNER = """
import os, sys
sys.path.insert(0, {root!r})
sys.path.insert(0, os.path.join({root!r}, "tests"))
from paper_2505_11204_b200 import randes, build
randes.LIB_PATH = {lib!r}
build.build_library = lambda *a, **k: randes.LIB_PATH
import pytest
rc = pytest.main(["-x", "-q", "-p", "no:cacheprovider", os.path.join({root!r}, "tests", "test_gpu_parity.py"), "-k",
                  "toy or ragged or mixed_group or more_tasks or unaligned or batched_retrieve_equals or adding_several or "
                  "large_and_partly or random_plans or multiples_of_eight"])
word, is_checked = randes.randes_debug_violation()
print("VIOLATION %d CHECKED %d" % (word, is_checked))
sys.exit(rc)
"""


def test_ordinary_build_reports_no_violation_and_says_what_it_is():
    build.build_library()
    assert randes.randes_debug_violation() == (0, False)


def test_parity_cases_pass_on_the_checked_build_without_a_violation(tmp_path):
    lib = str(tmp_path / "librandes_checked.so")
    subprocess.run(build.nvcc_command(lib, build.CHECKED_FLAGS), check=True)
    r = subprocess.run([sys.executable, "-c", RUNNER.format(root=ROOT, lib=lib)], capture_output=True, text=True, timeout=1800)
    assert r.returncode == 0, (r.stdout[-3000:], r.stderr[-3000:])
    assert "VIOLATION 0 CHECKED 1" in r.stdout, r.stdout[-2000:]
