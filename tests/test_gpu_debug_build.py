"""The checked build of the library (-DHEINSEN_DEBUG): compute-sanitizer is not available everywhere this library
runs, so the kernels can be compiled with their own index checks -- shared-memory window and alignment on every
access of the wrappers, element / row / tile / TMA coordinates in the kernels -- which record a failure and skip
the access instead of trapping.  This test builds that variant, runs small shapes through every kernel, staging
path and storage type in a process of its own, and requires correct results with no check fired."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_build_runs_clean(hs):
    from paper_2311_06281_b200 import build_ext
    lib = build_ext.build(debug=True)
    env = dict(os.environ, HEINSEN_SCAN_LIBRARY=lib)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_driver.py")], env=env, capture_output=True,
                       text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "no check fired" in r.stdout
    assert not hs.debug_build() and hs.debug_faults() is None     # the normal build has no checks and reports none
