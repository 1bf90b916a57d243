"""The bounds-checked build of the library (the stand-in for a memory checker): the same sources compiled with
-DPPOW_CHECKED test every kernel-computed index before use, count failures and skip the access (nothing traps).
Every GPU test of the suite is run against that library in a child pytest (PPOW_LIBRARY=checked); the child's
session fails if one check failed."""
import os
import subprocess
import sys

import pytest

from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import build as build_mod

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHECKED = os.environ.get("PPOW_LIBRARY") == "checked"


def test_ordinary_library_reports_that_it_is_not_the_checked_build():
    if CHECKED:
        pytest.skip("running against the checked build")
    assert B.ppow_checked_failures() == (B.PPOW_ERR_UNSUPPORTED, 0, 0)


@pytest.mark.skipif(not CHECKED, reason="only meaningful inside the child run against the checked build")
def test_checked_library_is_the_one_loaded_and_counts_nothing_so_far():
    status, failures, site = B.ppow_checked_failures()
    assert status == B.PPOW_OK and (failures, site) == (0, 0)


def test_every_gpu_test_passes_on_the_checked_build_without_a_failed_check():
    if CHECKED:
        pytest.skip("already inside the child run")
    build_mod.build(checked=True)
    env = dict(os.environ, PPOW_LIBRARY="checked")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", os.path.join(ROOT, "tests")]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=1800, env=env, cwd=ROOT)
    tail = res.stdout[-3000:] + res.stderr[-1000:]
    assert res.returncode == 0, tail
    assert "bounds-checked build: 0 failed checks" in res.stdout, tail
