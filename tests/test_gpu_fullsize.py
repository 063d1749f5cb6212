"""Full-size configurations in the launch configuration the benchmark times, checked on sampled outputs.

The oracle cannot finish these sizes in seconds, so it computes a seeded sample of (request, row, head)
units plus the boundary rows of the sampled requests.  Where the pools fit the host comfortably, KV append is
compared bit for bit over the whole pools; for the cells with a 131,072-token prefix (18 GB of K/V) the oracle
works request by request on the pages that request's block table names, and the appended pages of those
requests are compared bit for bit.  Inputs are generated on the device by the counter-based generators (same
bits as on the CPU).  Every-row checks at these sizes are in test_gpu_closed_forms.py.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests.helpers import bits, f64
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def boundary_rows(w, i):
    P, C = int(w.prefix_lens[i]), int(w.chunk_lens[i])
    cross = (-P) % w.page_size                      # first row that starts a new page
    rows = {0, 1, cross - 1, cross, 127, 128, 255, 256, C // 2, C - 2, C - 1}
    return sorted(r for r in rows if 0 <= r < C)


def sample_units(w, n_random, seed, heads_for_boundaries=(0, 1), max_boundary_requests=32, requests=None):
    """(request, row, head) triples: the boundary rows of the first requests plus seeded random units, all
    inside `requests` when given."""
    rng = np.random.default_rng(seed)
    units = []
    live = [i for i in (range(w.num_requests) if requests is None else requests) if w.chunk_lens[i] > 0]
    for i in live[:max_boundary_requests]:
        for t in boundary_rows(w, i):
            for h in heads_for_boundaries:
                units.append((i, t, min(h, w.num_q_heads - 1)))
            units.append((i, t, w.num_q_heads - 1))
    for _ in range(n_random):
        i = live[int(rng.integers(len(live)))]
        units.append((i, int(rng.integers(w.chunk_lens[i])), int(rng.integers(w.num_q_heads))))
    return np.array(units, dtype=np.int32)


def gather_units(w, res, units):
    rows = torch.from_numpy(w.q_offsets[units[:, 0]] + units[:, 1]).cuda()
    heads = torch.from_numpy(units[:, 2].astype(np.int64)).cuda()
    return f64(res["out"][rows, heads]), res["lse"][rows, heads].double().cpu().numpy()


def check_units(name, got, got_lse, ref, ref_lse, top2=None):
    keep = np.ones(len(ref), dtype=bool)
    if top2 is not None:
        # scores around 1e8 carry an fp32 error of tens of units: a row whose two largest scores are closer
        # than that has no well-defined answer in an fp32 pipeline; it is excluded and counted
        gap = top2[:, 0] - top2[:, 1]
        keep = gap >= (2.0 ** -18) * np.abs(top2[:, 0]) + 20.0
    assert keep.mean() > 0.95, f"too many ill-conditioned rows: {1 - keep.mean():.3f}"
    e = H.assert_close(got[keep], ref[keep], name)
    rel_lse = np.abs(got_lse[keep] - ref_lse[keep]) / np.maximum(1.0, np.abs(ref_lse[keep]))
    assert rel_lse.max() < 1e-3, rel_lse.max()
    e["excluded"] = int((~keep).sum())
    e["units"] = int(keep.sum())
    return e


def run_and_check_whole(w, units, opts=None, screen_ill_conditioned=False):
    """Whole pools on the host: append compared over every pool byte, attention on the sampled units."""
    dev = H.device_inputs(w)
    host = {k: v.cpu() for k, v in dev.items()}        # the generator's outputs, before the library touches them
    kp, vp = oracle.oracle_append(host["k_new"], host["v_new"], host["k_pool"], host["v_pool"], w.block_tables,
                                  w.prefix_lens, w.chunk_lens)
    del host["k_pool"], host["v_pool"]
    res = H.run_wave(w, dev, opts=opts)
    assert res["status"] == 0
    assert np.array_equal(bits(res["k_pool"]), kp), "K pool differs"
    assert np.array_equal(bits(res["v_pool"]), vp), "V pool differs"
    o = oracle.oracle_attention_units(host["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, units,
                                      return_top2=True)
    got, got_lse = gather_units(w, res, units)
    e = check_units(w.name, got, got_lse, o[0], o[1], o[2] if screen_ill_conditioned else None)
    assert not torch.isnan(res["out"].float()).any(), "a row was never written"
    e["plan"] = dict(tiles=int(res["plan"].info.num_tiles), split=int(res["plan"].info.num_split_tiles))
    return e


def run_and_check_sliced(w, requests, n_random, seed, opts=None):
    """Pools stay on the device: the oracle runs request by request on the pages the request's table names."""
    dev = H.device_inputs(w)
    slices = {i: H.request_slice(w, dev, i) for i in requests}      # before the wave: the append writes those pages
    res = H.run_wave(w, dev, opts=opts)
    assert res["status"] == 0
    units = sample_units(w, n_random, seed, max_boundary_requests=len(requests), requests=requests)
    got, got_lse = gather_units(w, res, units)
    ref = np.empty_like(got)
    ref_lse = np.empty_like(got_lse)
    for i, sl in slices.items():
        kp, vp = oracle.oracle_append(sl["k_new"], sl["v_new"], sl["k_pool"], sl["v_pool"], sl["block_tables"],
                                      sl["prefix_lens"], sl["chunk_lens"])
        gk, gv = H.appended_pages_of(dev, sl)
        assert np.array_equal(bits(gk), kp), f"K pages of request {i} differ"
        assert np.array_equal(bits(gv), vp), f"V pages of request {i} differ"
        sel = np.nonzero(units[:, 0] == i)[0]
        u = units[sel].copy()
        u[:, 0] = 0
        o, l = oracle.oracle_attention_units(sl["q"], kp, vp, sl["block_tables"], sl["prefix_lens"], sl["chunk_lens"], u)
        ref[sel], ref_lse[sel] = o, l
    e = check_units(w.name, got, got_lse, ref, ref_lse)
    assert not torch.isnan(res["out"].float()).any(), "a row was never written"
    assert not torch.isnan(res["lse"]).any()
    e["plan"] = dict(tiles=int(res["plan"].info.num_tiles), split=int(res["plan"].info.num_split_tiles))
    return e


def test_cfg3_concurrency_128_high_reuse():
    w = W.cfg3()
    print("cfg3", run_and_check_whole(w, sample_units(w, 6000, seed=303)))


@pytest.mark.parametrize("splits", [0, 4])
def test_cfg4_long_context_alternating_scale(splits):
    w = W.cfg4("alternate")
    e = run_and_check_whole(w, sample_units(w, 3000, seed=404, max_boundary_requests=3), opts=wpp.PlanOpts(0, 0, splits, 0))
    assert (e["plan"]["split"] > 0) == (splits > 0)
    print("cfg4_alt", splits, e)


@pytest.mark.parametrize("splits,rescale_mode", [(0, 0), (8, 0), (0, 1)])
def test_cfg4_long_context_cumulative_scale(splits, rescale_mode):
    """K doubles every 4096 positions (up to 2^25): the running reference jumps 26 times per row.  Both orders of
    work of the kernel (accumulator rescaled before or after the step's exponentials) are checked."""
    w = W.cfg4("cumulative")
    H.ctx().set_rescale_mode(rescale_mode)
    try:
        e = run_and_check_whole(w, sample_units(w, 3000, seed=405, max_boundary_requests=3),
                                opts=wpp.PlanOpts(0, 0, splits, 0), screen_ill_conditioned=True)
    finally:
        H.ctx().set_rescale_mode(0)
    print("cfg4", splits, rescale_mode, e)


CHUNKS = (64, 256, 1024, 4096, 8192)
PREFIXES = (0, 4096, 32768, 131072)


@pytest.mark.parametrize("P", PREFIXES)
@pytest.mark.parametrize("C", CHUNKS)
def test_cfg5_sweep_cells(C, P):
    """All twenty cells of the sweep grid at the stated batch of 32 requests."""
    w = W.cfg5_cell(C, P, num_requests=32)
    if P <= 32768:
        e = run_and_check_whole(w, sample_units(w, 400, seed=505 + C + P, max_boundary_requests=4))
    else:
        e = run_and_check_sliced(w, requests=(0, 13, 31), n_random=300, seed=505 + C + P)
    print(w.name, e)
