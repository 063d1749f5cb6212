"""The tile ring of the attention kernel gives up one K slot when the alignment of the shared-memory base leaves
too little room.  That fallback does not occur on the boxes at hand, so a library built with
WPP_FORCE_SMALL_RING takes it always, and a child process checks that build against the oracle."""
import os
import subprocess
import sys
import tempfile

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r})
import numpy as np
import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests.helpers import cpu_inputs, f64, run_oracle
from tests import gpu_harness as H
cases = [
    W.custom_workload([300, 0, 1000, 64], [17, 260, 3, 128], 8, 2, 128, 64, seed=7, spare_pages=5),
    W.custom_workload([1500] * 6, [700] * 6, 8, 2, 128, 64, seed=9),          # long tile lists, unequal halves
    W.custom_workload([5, 130, 257], [400, 1, 127], 4, 4, 64, 32, seed=7),
]
for w in cases:
    inp = cpu_inputs(w)
    kp, vp, ref, ref_lse = run_oracle(w, inp)
    for opts in (wpp.PlanOpts(256, 0, 0, 3), wpp.PlanOpts(128, 0, 0, 0)):
        res = H.run_wave(w, H.device_inputs(w, inp), opts=opts)
        assert res["status"] == 0, res["status"]
        H.assert_close(f64(res["out"]), ref, w.name)
print("small ring ok")
"""


def test_small_ring_build_matches_oracle():
    from paper_2609_35263_b200 import build as B
    with tempfile.TemporaryDirectory() as tmp:
        lib = os.path.join(tmp, "libwpp_small_ring.so")
        B.build(defines=["WPP_FORCE_SMALL_RING"], out=lib)
        env = dict(os.environ, WPP_LIB_PATH=lib)
        r = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], env=env, capture_output=True, text=True,
                           timeout=600)
        assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
        assert "small ring ok" in r.stdout
