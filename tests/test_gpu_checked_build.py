"""The bounds-checked build of the CUDA library on the small and ragged cases (needs a B200).

compute-sanitizer is not available on this machine, so the library can be compiled a second time with
-DTOPOEP_CHECKED: every index that is derived from data (expert ids read from records, instance
ids, list positions, work-list entries) is checked; a bad one sets TOPOEP_FLAG_INTERNAL and is
clamped, nothing traps.  A process loads one build of the library, so the cases run in a child
process with TOPOEP_CHECKED_BUILD=1 (tests/checked_cases.py).
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_build_runs_the_small_cases_without_a_single_bad_index():
    env = dict(os.environ, TOPOEP_CHECKED_BUILD="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "checked_cases.py")], env=env,
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "no index check fired" in res.stdout
