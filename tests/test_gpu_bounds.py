"""The bounds-checking build stands in for a memory checker: the same cases as the normal parity
tests (tiny, decode steps over tile edges on both kernels, units finished inside the kernel, a batch
below the capacity, evicted slots, replays past the capacity, prefill) run against a library compiled
with -DKVS_DEBUG_BOUNDS, in which every computed global offset is checked on the device, with canary
patterns around the pool and in every row no token may occupy."""
import os
import subprocess
import sys

import pytest

from paper_2410_18517_b200 import build as kbuild

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_cases_under_the_bounds_checking_build():
    lib = kbuild.build(bounds=True)
    env = dict(os.environ, KVS_LIBRARY=lib, PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests")]))
    out = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "bounds_cases.py")], capture_output=True, text=True,
                         timeout=1500, env=env)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-3000:]
    assert "ALL BOUNDS CASES PASSED" in out.stdout
