"""The small GPU parity cases once more under the bounds-checking build of the library.

compute-sanitizer is not available on the machines these tests run on, so out-of-range indexing is looked for with the
library's own second build (-DBEAGLE_BOUNDS_CHECK): every cache scatter, chunk read and token gather whose index comes
from the host's per-call metadata is checked on the device against the extent the kernel was given; a violation raises the
context's device error word (the access is skipped, nothing traps) and the autouse fixture of conftest.py, which asks every
open context for its device status after each test, fails the test.  Valid inputs only: what is shown is that no check fires.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def test_small_parity_cases_pass_under_the_bounds_checking_build():
    if os.environ.get("BEAGLE_LIBRARY"):
        pytest.skip("already running under an alternative build of the library")
    from paper_2505_24544_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, BEAGLE_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join("tests", "test_parity_gpu.py"), "-x", "-m", "gpu"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    tail = r.stdout[-3000:] + r.stderr[-1000:]
    assert "bounds-checking build" in r.stdout, tail          # the child really loaded the checked library
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "failed" not in r.stdout.splitlines()[-1], tail
