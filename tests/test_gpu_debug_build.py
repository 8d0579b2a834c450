"""The bounds-checked build (-DZC_DEBUG): its kernels check the indices they address tiles,
rows and partials with and report the first failed check through zc_device_status.  A set of
parity cases is run against it in a process of its own (the library is loaded once per
process); all checks must pass."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_parity_cases_pass_every_index_check_of_the_debug_build():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "helpers", "run_debug_build.py")],
                         capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "debug build ok" in res.stdout
