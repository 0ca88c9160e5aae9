"""The bounds-checked build of the library (libloki_alloc_debug.so, the sources compiled with
-DLOKI_DEBUG): every index into the device tables, the shared-memory stages and tables of the
scoring kernels and the partial-key scratch is checked inside the kernels, a violation is
recorded in the handle's status words and the index replaced by a valid one -- nothing traps and
nothing faults.  The test runs the small named workloads and random problems through every
scoring kernel of that build in a process of its own, wants the oracle's plans, and wants the
status words clean.  It stands in for a memory checker on machines where none can be run."""
import json
import os
import subprocess
import sys

import pytest

from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import build as lib_build

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def test_checked_build_runs_clean_and_matches_the_oracle():
    lib = lib_build.DEBUG_LIB_PATH
    if not os.path.exists(lib):
        lib = lib_build.build_library(debug=True)
    env = dict(os.environ, LOKI_ALLOC_LIB=lib)
    r = subprocess.run([sys.executable, os.path.join(HERE, "debug_build_driver.py")], env=env,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    out = json.loads(r.stdout.strip().splitlines()[-1])
    assert out["checked_build"] == 1
    assert out["n_solves"] >= 100 and out["n_mismatch"] == 0
    assert out["site_mask"] == 0 and out["n_violations"] == 0


def test_release_build_reports_that_it_checks_nothing():
    from paper_2407_03583_b200 import workloads as W
    a = B.Allocator(W.make_workload("C1"))
    try:
        a.solve(W.make_workload("C1").demand_mqps)
        assert B.loki_alloc_debug_status(a.handle) == (0, 0, 0)
    finally:
        a.close()
