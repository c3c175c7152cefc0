"""The small-shape parity tests once more under the checked build of the library
(libsnapstream_dbg.so, compiled with -DSNAP_DEBUG_BOUNDS): every data-dependent index -- selected
positions, output ranks, ring slots, band entries, corrected ranks -- is tested against its
array, a bad one raises SNAP_DEV_INDEX_CHECK in the status word (which the parity tests require
to be zero) and the access is skipped.  Stands in for a memory checker, without ever trapping."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_shape_parity_under_the_checked_build():
    from paper_2511_03092_b200 import build as snap_build
    lib = snap_build.build(debug_bounds=True)
    assert os.path.exists(lib)
    env = dict(os.environ, SNAP_LIBRARY=os.path.basename(lib))
    cmd = [sys.executable, "-m", "pytest", "tests/test_gpu_parity.py", "tests/test_gpu_near_ties.py", "-m", "gpu", "-q", "-x",
           "-p", "no:cacheprovider"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
