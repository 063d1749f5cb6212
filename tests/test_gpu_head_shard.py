"""KV-head sharding of the attention calls (the first half of the step after the hot path): two shards, run one
after the other on one GPU through strided views of the same tensors, must reproduce the unsharded result - pools
bit for bit, outputs bit for bit when neither run splits keys, and within tolerance of the oracle in any case."""
import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from paper_2609_35263_b200.stages import head_shard
from tests import gpu_harness as H
from tests.helpers import bits, cpu_inputs, f64, run_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world,force_splits", [(2, 1), (4, 1), (2, 0)])
def test_head_shards_reproduce_the_unsharded_wave(world, force_splits):
    w = W.custom_workload([300, 0, 1000, 64], [200, 260, 3, 130], 16, 4, 128, 64, seed=21)
    inp = cpu_inputs(w)
    kp_ref, vp_ref, ref, _ = run_oracle(w, inp)
    opts = wpp.PlanOpts(0, 0, force_splits, 0)
    whole = H.run_wave(w, H.device_inputs(w, inp), opts=opts)
    assert whole["status"] == 0

    dev = torch.device("cuda")
    g = H.device_inputs(w, inp)
    out = torch.empty(w.total_new_tokens, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    out.view(torch.int16).fill_(0x7FC0)
    bt = torch.from_numpy(w.block_tables).to(dev)
    P, C = torch.from_numpy(w.prefix_lens).to(dev), torch.from_numpy(w.chunk_lens).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for rank in range(world):
        d, v = head_shard(rank, world, w.num_requests, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size,
                          w.max_blocks_per_req, w.num_pages, g["q"], out, g["k_new"], g["v_new"], g["k_pool"], g["v_pool"])
        assert d.num_kv_heads == w.num_kv_heads // world and d.num_q_heads == w.num_q_heads // world
        plan = wpp.wpp_plan_tiles(H.ctx(), d, w.prefix_lens, w.chunk_lens, opts=opts).to_device()
        ws = torch.empty(max(256, int(plan.info.workspace_bytes)), dtype=torch.uint8, device=dev)
        wpp.wpp_kv_append(H.ctx(), d, v["k_new"], v["v_new"], v["k_pool"], v["v_pool"], bt, P, C, plan, status=status)
        wpp.wpp_prefill_attention_varlen(H.ctx(), d, v["q"], v["out"], None, v["k_pool"], v["v_pool"], bt, P, C, plan,
                                         workspace=ws, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(bits(g["k_pool"]), kp_ref) and np.array_equal(bits(g["v_pool"]), vp_ref)
    H.assert_close(f64(out), ref, f"{world} head shards")
    if force_splits == 1:
        assert torch.equal(out.view(torch.int16), whole["out"].view(torch.int16))


def test_uneven_shards_are_refused():
    t = torch.zeros(4, 6, 8)
    with pytest.raises(ValueError):
        head_shard(0, 4, 1, 6, 6, 8, 16, 1, 1, t, t, t, t, t.unsqueeze(2), t.unsqueeze(2))
