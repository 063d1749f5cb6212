"""The entry point that allocates nothing (collected last on purpose).

Some callers of this library cannot allocate device memory when a wave is due: the serving process has given
every free byte of HBM to the KV page pool, and cudaMalloc on the execution stream would fail or stall it.  For
them the library keeps a fixed scratch array for the split-KV partials.  This test calls that entry point through
the C ABI twice in a row and checks it against the caller-workspace entry point and against the fp64 oracle, and
that the free device memory is the same before and after a call; it must pass alone in a fresh process as well as
after every other test.
"""
import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests import gpu_harness as H
from tests.helpers import cpu_inputs, f64, run_oracle

pytestmark = pytest.mark.gpu


def _setup(w, splits, inp=None):
    c = H.ctx()
    d = H.desc_of(w)
    dev = H.device_inputs(w, inp)
    plan = wpp.wpp_plan_tiles(c, d, w.prefix_lens, w.chunk_lens, opts=wpp.PlanOpts(0, 0, splits, 0)).to_device()
    meta = [torch.from_numpy(x).cuda() for x in (w.block_tables, w.prefix_lens, w.chunk_lens)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    wpp.wpp_kv_append(c, d, dev["k_new"], dev["v_new"], dev["k_pool"], dev["v_pool"], *meta, plan, status=status)
    return c, d, dev, plan, meta, status


def test_static_scratch_entry_point_matches_the_workspace_entry_point_twice():
    w = W.custom_workload([900, 0, 130, 4000], [300, 500, 64, 200], 4, 2, 128, 64, seed=31)
    inp = cpu_inputs(w)
    _, _, oracle_out, oracle_lse = run_oracle(w, inp)
    c, d, dev, plan, meta, status = _setup(w, splits=3, inp=inp)
    assert 0 < plan.info.workspace_bytes <= wpp.wpp_static_scratch_bytes()
    T = w.total_new_tokens
    shape = (T, w.num_q_heads, w.head_dim)
    ref = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    ref_lse = torch.empty(T, w.num_q_heads, dtype=torch.float32, device="cuda")
    ws = torch.empty(int(plan.info.workspace_bytes), dtype=torch.uint8, device="cuda")
    wpp.wpp_prefill_attention_varlen(c, d, dev["q"], ref, ref_lse, dev["k_pool"], dev["v_pool"], *meta, plan,
                                     workspace=ws, status=status)
    torch.cuda.synchronize()
    for call in range(2):
        out = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((T, w.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        wpp.wpp_prefill_attention_varlen_static(c, d, dev["q"], out, lse, dev["k_pool"], dev["v_pool"], *meta, plan,
                                                status=status)
        torch.cuda.synchronize()
        # the context looked the scratch array up when it was created, so not even the first call places anything
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
        assert int(status.item()) == 0
        H.assert_close(f64(out), oracle_out, f"static entry point, call {call}")
        assert np.abs(lse.double().cpu().numpy() - oracle_lse).max() < 2e-2
        diff = (out.double() - ref.double()).abs()
        assert not torch.isnan(out.float()).any()
        assert diff.max().item() <= H.MAX_ABS_TOL and diff.mean().item() <= H.MEAN_ABS_TOL, (call, diff.max().item())
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16)), "same plan, same kernels: same bits"
        assert torch.allclose(lse, ref_lse, atol=1e-6)


def test_static_scratch_entry_point_rejects_plans_beyond_its_limit():
    w = W.custom_workload([16384] * 16, [512] * 16, 16, 2, 128, 64, seed=32)
    c, d, dev, plan, meta, status = _setup(w, splits=16)
    assert plan.info.workspace_bytes > wpp.wpp_static_scratch_bytes()
    out = torch.empty(w.total_new_tokens, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    launches = c.launch_count()
    with pytest.raises(wpp.WppError) as e:
        wpp.wpp_prefill_attention_varlen_static(c, d, dev["q"], out, None, dev["k_pool"], dev["v_pool"], *meta, plan,
                                                status=status)
    assert e.value.status == 5 and c.launch_count() == launches       # WPP_ERR_WORKSPACE_TOO_SMALL, nothing launched
