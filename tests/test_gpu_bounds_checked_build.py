"""The bounds-checking build of the library (the stand-in for a memory checker, which is not
available here): compiled with -DINSTINFER_BOUNDS_CHECK, every data-dependent global offset a
kernel computes is tested against the extent the call's shapes imply, and a violation sets
status bit 8 instead of being used.  The small ragged / paged / sparse / grouped / bulk-append
parity cases are run against that build in a child process; every one of them asserts that
the status word stays 0, so a single stray offset anywhere fails the run."""
import os
import subprocess
import sys

import pytest

from paper_2409_04992_b200 import build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = ["tests/test_gpu_parity_small.py", "tests/test_gpu_invariants.py", "tests/test_gpu_sparf.py",
         "tests/test_gpu_grouped.py", "tests/test_gpu_bulk_append.py", "tests/test_gpu_head_sharded.py"]


def test_small_cases_raise_no_bounds_flag_in_the_checked_build():
    library = build.build(checked=True)
    env = dict(os.environ, INSTINFER_LIBRARY=str(library))
    done = subprocess.run([sys.executable, "-m", "pytest", *CASES, "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider"],
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=1800)
    assert done.returncode == 0, done.stdout[-4000:] + done.stderr[-2000:]
    assert " passed" in done.stdout
