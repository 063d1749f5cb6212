"""Seeded random ragged waves against the oracle: shapes, head ratios, page sizes, planner options and the number of
persistent CTAs all vary, so that corner combinations no hand-written case lists still get exercised."""
import numpy as np
import pytest

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests.test_gpu_parity import _full_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(64))
def test_random_ragged_wave(seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    B = int(rng.choice([16, 32, 64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 3, 4, 8]))
    R = int(rng.integers(1, 7))
    P = [int(x) for x in rng.choice([0, 1, B - 1, B, 3 * B + 5, 130, 257, 700], R)]
    C = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 127, 128, 129, 300, 401], R)]
    if sum(C) == 0:
        C[0] = 33
    w = W.custom_workload(P, C, Hkv * G, Hkv, d, B, seed=seed, spare_pages=int(rng.integers(1, 6)))
    opts = wpp.PlanOpts(int(rng.choice([0, 128, 256])), 0, int(rng.choice([0, 0, 1, 2, 3])),
                        int(rng.choice([0, 1, 2, 5, 37, 148])), int(rng.integers(0, 2)))
    _full_parity(w, opts=opts)            # both kernel shapes
