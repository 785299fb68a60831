"""The checked build of the library (compiled with -DPF_BOUNDS_CHECK: every index into a shared-memory image, queue,
table, timeline, order table, key list or output array is range-checked on the device; a violation sets a bit in the
plan's check record and the access is redirected, nothing traps).  It stands in for a memory checker: the small
spaces, eight randomized spaces, sub-ranges, the one-call search, the selection, the compact view, the
deep-pipeline simulator cases and a 9.7e7-candidate search that splits its work over the plan's streams must all leave the record empty.  Runs in a process of its own so that the checked
library never mixes with the ordinary one."""
from __future__ import annotations

import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))


def test_checked_build_reports_no_bad_index():
    from paper_2607_18631_b200 import build as pf_build
    lib = pf_build.build(bounds_check=True)
    env = dict(os.environ, PLANFRONT_LIB=lib)
    r = subprocess.run([sys.executable, os.path.join(HERE, "checked_build_run.py")], env=env, capture_output=True,
                       text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    lines = [ln for ln in r.stdout.splitlines() if " status=" in ln]
    assert len(lines) == 2 + 4 + 8 + 1 + 1, r.stdout
    # the macro does record a bad index: site 17 (bit 131072), index 7, length 4 -- and reading clears the record
    assert lines[0] == "selftest status=0 record=131072 17 7 0 4 0", lines[0]
    assert lines[1] == "selftest_cleared status=0 record=0 0 0 0 0 0", lines[1]
    for ln in lines[2:]:
        # status 0: this IS the checked build (the ordinary one answers PF_EUNSUPPORTED); record all zero: clean
        assert ln.split(" status=")[1] == "0 record=0 0 0 0 0 0", ln


def test_ordinary_build_has_no_checks():
    import numpy as np
    from paper_2607_18631_b200 import Plan
    from paper_2607_18631_b200.binding import PF_EUNSUPPORTED
    from workloads import make_config
    if os.environ.get("PLANFRONT_LIB"):
        pytest.skip("another library build was selected")
    plan = Plan(make_config("tiny"))
    st, rec = plan.check_read()
    assert st == PF_EUNSUPPORTED and not np.any(rec)
    plan.close()
