"""The bounds-checking debug build of the library (every global access of the streaming kernels
checked against the work item it belongs to and the vector, every scratch index against its
table; violations counted and skipped) on ragged problems: the kernels must not attempt a single
access outside their own item.  This stands in for a memory checker."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_no_out_of_range_access_on_ragged_problems():
    env = dict(os.environ, GRAWA_DEBUG_BOUNDS="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_bounds_cases.py")], env=env,
                         capture_output=True, text=True, timeout=1200)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    out = json.loads(res.stdout.strip().splitlines()[-1])
    assert out["selfcheck"] == 7          # the checker itself counts (seven planted violations, two clean probes)
    assert out["cases"] > 300
    assert out["violations"] == 0


def test_normal_build_reports_that_it_does_not_check():
    import paper_2403_04206_b200 as grawa
    if os.environ.get("GRAWA_DEBUG_BOUNDS") == "1":
        pytest.skip("debug build selected")
    assert grawa.grawa_debug_bounds_violations() == -1
