"""The tuned kernels under the bounds-checking build of the library (-DSSM_DEBUG_BOUNDS): every tile row index and every
global row / channel offset they store to is range-checked on the device, a violation is clamped or skipped and reported
by ssm_scan_check_status as SSM_ERR_BOUNDS.  Nothing traps, so this is safe to run on a shared GPU; it stands in for a
memory checker on small shapes with ragged tiles, partial channel groups and time splits."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shapes_under_bounds_checking_build():
    from paper_2312_00752_b200 import build as B
    lib = B.build_library(debug_bounds=True) if not os.path.exists(B.DEBUG_LIB_PATH) else B.DEBUG_LIB_PATH
    env = dict(os.environ, SSM_SCAN_LIBRARY=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-m", "tests._debug_bounds_worker"], cwd=ROOT, env=env, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-3000:]
    assert "no index left its range" in res.stdout
