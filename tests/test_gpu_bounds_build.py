"""GPU: the checked build of the library (-DSURGEON_BOUNDS) on a small list of shapes.  A memory
checker cannot be run on these GPUs, so the library carries its own: in that build every guarded
global store (packed values of the compaction, partial tiles of the weight gradient) tests its
index against the size the host computed, records SURGEON_ERR_INTERNAL and skips the store when it
lies outside.  The worker runs in a child process that loads the checked build."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_build_matches_the_oracle_and_reports_no_index_out_of_bounds():
    from paper_2503_20354_b200 import build
    lib = build.build(bounds=True)
    env = dict(os.environ, SURGEON_LIB=lib)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "bounds_worker.py")], env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "BOUNDS_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-3000:]
