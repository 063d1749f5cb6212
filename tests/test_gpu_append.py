"""KV append alone: bit-exact against the oracle over the entire pools, including odd bit patterns."""
import numpy as np
import pytest
import torch

import oracle
import wpp_workloads as W
from tests.helpers import bits, cpu_inputs, from_bits
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("P,C,Hkv,d,B", [
    ([0], [1], 1, 64, 16),
    ([37, 0, 129], [200, 1, 64], 2, 128, 16),
    ([5, 130, 257, 0], [400, 1, 127, 0], 4, 64, 32),
    ([4096], [3000], 8, 128, 64),
    ([1, 2, 3], [300, 300, 300], 2, 128, 128),
])
def test_append_is_bit_exact(P, C, Hkv, d, B):
    w = W.custom_workload(P, C, Hkv * 2, Hkv, d, B, seed=21, spare_pages=7)
    inp = cpu_inputs(w)
    kn = bits(inp["k_new"]).copy()
    if kn.size >= 4:
        kn.reshape(-1)[:4] = [0x7FC1, 0x8000, 0xFF80, 0xFFFF]      # NaN payload, -0, -inf, NaN
    inp["k_new"] = from_bits(kn)
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"], w.block_tables,
                                  w.prefix_lens, w.chunk_lens)
    res = H.run_wave(w, H.device_inputs(w, inp), do_attention=False)
    assert res["status"] == 0
    assert np.array_equal(bits(res["k_pool"]), kp)
    assert np.array_equal(bits(res["v_pool"]), vp)


def test_append_shared_prefix_pages_are_left_alone():
    rng = np.random.default_rng(22)
    w = W.make_workload("shared", 22, rng, [128, 150, 128], [64, 10, 100], 4, 2, 128, 64, shared_tokens=128,
                        sharers=[True, True, True], spare_pages=3)
    inp = cpu_inputs(w)
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"], w.block_tables,
                                  w.prefix_lens, w.chunk_lens)
    res = H.run_wave(w, H.device_inputs(w, inp), do_attention=False)
    assert np.array_equal(bits(res["k_pool"]), kp) and np.array_equal(bits(res["v_pool"]), vp)
    shared = w.block_tables[0, :2]
    assert np.array_equal(bits(res["k_pool"])[shared], bits(inp["k_pool"])[shared])
