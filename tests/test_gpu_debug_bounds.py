"""The bounds-checking build of the library (-DDAB_DEBUG_BOUNDS: every global-memory index of the hot-path kernels
compared with the extent of its array) must report no violation over ragged shapes, all coders and both contraction
kernels.  It runs in a process of its own because a process loads one build of the library."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_debug_bounds_build_reports_no_violation():
    from paper_1804_02941_b200 import build
    lib = build.build(debug_bounds=True)    # compiles only if a source is newer than libdab_debug.so
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_bounds_run.py"), lib], capture_output=True,
                       text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    report = json.loads(r.stdout.strip().splitlines()[-1])
    assert report["calls"] > 100 and report["compared"] == 4
    assert report["violations"] == 0, report
    assert report["wait_failures"] == 0


def test_ordinary_build_has_no_checks():
    import paper_1804_02941_b200 as dab
    assert not dab.dab_debug_bounds_enabled()
    with pytest.raises(dab.DabError) as e:
        dab.dab_debug_bounds_report()
    assert e.value.status == 2
