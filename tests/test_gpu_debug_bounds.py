"""The checked build (libks_debug.so, KS_DEBUG_BOUNDS): the quantised tree kernels compare every
index they form from data (tile byte, node, chunk, record, memo slot, partial list) with its
range and record the first violation instead of touching memory out of range. The small parity
cases of tests/debug_bounds_cases.py must pass on it with the word still 0. This stands in for a
memory checker, which this machine pool does not offer."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_small_cases_on_the_checked_build():
    from paper_2609_35587_b200 import build
    lib = build.build(debug=True)
    env = dict(os.environ, KS_LIBRARY=lib, PYTHONPATH=ROOT)
    r = subprocess.run([sys.executable, "-m", "tests.debug_bounds_cases"], cwd=ROOT, env=env,
                       capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-3000:]
    assert "no index out of range" in r.stdout


def test_regular_build_reports_no_checked_build():
    """Without a GPU: the symbol exists and the regular library answers -1 ... only where a
    device is present (the call synchronises); here only the export is checked."""
    import ctypes
    from paper_2609_35587_b200 import build
    lib = ctypes.CDLL(build.build())
    assert hasattr(lib, "ks_debug_bounds_line") and hasattr(lib, "ks_debug_set_wait")
