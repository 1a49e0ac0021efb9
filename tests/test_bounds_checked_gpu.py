"""The range-checked build of the library (-DSD_BOUNDS_CHECK: every index the kernels form into global
memory is tested against its extent; a failing access is skipped and counted) runs every entry point on
tiny, ragged and multi-stage shapes, agrees with the oracle, and counts no violation.  It stands in for a
memory checker: the tool itself is not available for these runs."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_checked_build_counts_no_violation():
    import __graft_entry__ as entry
    entry.build()
    assert os.path.exists(entry.LIB_CHECKED)
    env = dict(os.environ, SD_VERIFY_LIBRARY=entry.LIB_CHECKED,
               PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests"), os.environ.get("PYTHONPATH", "")]))
    run = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "checked_build_runner.py")], env=env, cwd=ROOT,
                         capture_output=True, text=True, timeout=1200)
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-3000:]
    line = [ln for ln in run.stdout.splitlines() if ln.startswith("REPORT ")][-1]
    report = json.loads(line[len("REPORT "):])
    assert report == {"violations": 0, "site": 0, "index": 0, "limit": 0}, report


def test_regular_build_says_it_has_no_checks():
    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding
    if not os.environ.get("SD_VERIFY_LIBRARY"):
        assert binding.sd_bounds_report() is None
