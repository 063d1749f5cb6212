"""GPU parity: the CUDA path through the C ABI against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests.helpers import bits, cpu_inputs, f64, from_bits, run_oracle
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def _full_parity(w, opts=None, inp=None, sm_scale=0.0, shapes=(1, 2)):
    """Both attention kernel shapes (unless the options name one) against the oracle; returns the last run."""
    inp = inp or cpu_inputs(w)
    kp, vp, ref, ref_lse = run_oracle(w, inp, sm_scale=sm_scale or None)
    if opts is not None and opts.shape:
        shapes = (opts.shape,)
    for shape in shapes:
        res = H.run_wave(w, H.device_inputs(w, inp), opts=opts, sm_scale=sm_scale, shape=shape)
        assert res["status"] == 0 and res["plan"].info.shape == shape
        # append and page indexing: bit exact over the whole pools
        assert np.array_equal(bits(res["k_pool"]), kp), "K pool differs"
        assert np.array_equal(bits(res["v_pool"]), vp), "V pool differs"
        e = H.assert_close(f64(res["out"]), ref, f"{w.name} shape {shape}")
        lse = res["lse"].double().cpu().numpy()
        assert np.isfinite(lse).all() and np.abs(lse - ref_lse).max() < 2e-2, np.abs(lse - ref_lse).max()
    return res, e


@pytest.mark.parametrize("tile_m", [0, 128, 256])
def test_cfg1_single_request(tile_m):
    res, e = _full_parity(W.cfg1(), opts=wpp.PlanOpts(tile_m, 0, 0, 0))
    print("cfg1", e)


def test_odd_group_size_leaves_single_halves():
    """Three query heads per KV head: short tails cannot be paired, so tiles with one unused half appear."""
    w = W.custom_workload([40, 300], [70, 130], 3, 1, 128, 64, seed=18)
    _full_parity(w, opts=wpp.PlanOpts(256, 0, 0, 0))
    _full_parity(w, opts=wpp.PlanOpts(256, 0, 2, 0))


@pytest.mark.parametrize("P,C,Hq,Hkv,d,B", [
    ([0], [1], 2, 1, 64, 16),                    # one key: output is V[0] exactly
    ([0], [128], 4, 2, 128, 64),                 # pure causal, exactly one tile
    ([0], [129], 2, 2, 128, 64),                 # one row spills into a second tile
    ([37], [200], 4, 1, 128, 16),                # prefix ends mid page and mid key step
    ([300, 0, 1000, 64], [17, 260, 3, 128], 8, 2, 128, 64),
    ([5, 130, 257], [400, 1, 127], 4, 4, 64, 32),
    ([1024], [512], 2, 1, 128, 128),
    ([100, 0], [0, 70], 2, 1, 64, 16),           # an empty chunk in the wave
])
@pytest.mark.parametrize("tile_m", [128, 256])
def test_ragged_small(P, C, Hq, Hkv, d, B, tile_m):
    w = W.custom_workload(P, C, Hq, Hkv, d, B, seed=7, spare_pages=5)
    _full_parity(w, opts=wpp.PlanOpts(tile_m, 0, 0, 0))


@pytest.mark.parametrize("C,Hq,Hkv,d,B", [
    ([1, 7, 16], 16, 2, 128, 64),        # eight heads of a KV group packed into one 128-row half
    ([17, 32, 3], 8, 2, 128, 64),        # four heads per half
    ([33, 64, 40], 8, 1, 128, 16),       # two heads per half, second half takes the next two
    ([64, 5], 8, 2, 64, 16),
    ([20, 50], 6, 1, 128, 64),           # group of six: packs of two
])
@pytest.mark.parametrize("splits", [0, 2])
def test_short_chunks_pack_heads(C, Hq, Hkv, d, B, splits):
    P = [300, 0, 129][:len(C)]
    w = W.custom_workload(P, C, Hq, Hkv, d, B, seed=19, spare_pages=4)
    res, _ = _full_parity(w, opts=wpp.PlanOpts(256, 0, splits, 0))
    _full_parity(w, opts=wpp.PlanOpts(128, 0, splits, 0))


@pytest.mark.parametrize("tile_m,splits,ctas", [(256, 2, 3), (128, 3, 2), (256, 1, 1), (128, 1, 5)])
def test_many_tiles_per_cta_back_to_back(tile_m, splits, ctas):
    """Few persistent CTAs walk long tile lists: a tile's first product must not overwrite the accumulator
    while the previous tile's epilogue (slow for fp32 partials) is still reading it."""
    w = W.custom_workload([700, 0, 260, 64], [200, 300, 64, 129], 8, 2, 128, 64, seed=23, spare_pages=4)
    _full_parity(w, opts=wpp.PlanOpts(tile_m, 0, splits, ctas))


@pytest.mark.parametrize("ctas", [1, 2, 7])
def test_single_step_tiles_back_to_back(ctas):
    """Tiles of one key step, many per CTA: the softmax warps could finish tile k+1 before the epilogue has
    consumed tile k's end-of-tile values; the hand-over must hold them back (repeated to catch a race)."""
    w = W.custom_workload([0, 0, 10, 0, 60, 0], [64, 128, 100, 33, 68, 1], 16, 2, 128, 64, seed=24, spare_pages=4)
    inp = cpu_inputs(w)
    _, _, ref, _ = run_oracle(w, inp)
    first = None
    for rep in range(6):
        res = H.run_wave(w, H.device_inputs(w, inp), opts=wpp.PlanOpts(256 if rep % 2 else 128, 0, 1, ctas), shape=1 + rep % 2 if rep < 4 else None)
        assert res["status"] == 0
        H.assert_close(f64(res["out"]), ref, f"single-step tiles, {ctas} CTAs, repeat {rep}")


@pytest.mark.parametrize("shape", [1, 2])
def test_single_key_is_bit_exact(shape):
    w = W.custom_workload([0], [1], 4, 2, 128, 64, seed=8)
    inp = cpu_inputs(w)
    res = H.run_wave(w, H.device_inputs(w, inp), shape=shape)
    v0 = inp["v_new"][0]                                     # [Hkv, d]
    out = res["out"].cpu()
    for h in range(4):
        assert torch.equal(out[0, h].view(torch.int16), v0[h // 2].view(torch.int16))


@pytest.mark.parametrize("tile_m", [128, 256])
@pytest.mark.parametrize("splits", [2, 3, 7])
def test_forced_kv_splits_and_combine(splits, tile_m):
    w = W.custom_workload([900, 0, 130], [300, 500, 64], 4, 2, 128, 64, seed=9)
    opts = wpp.PlanOpts(tile_m, 0, splits, 0)
    res, _ = _full_parity(w, opts=opts)
    assert res["plan"].info.num_combine_tiles > 0 and res["plan"].info.workspace_bytes > 0


def test_tail_round_cut_along_the_keys_by_the_planner():
    """Eight long tiles on six CTAs: the planner cuts the two tiles of the second round in three (nobody asked for
    splits: six parts fill the six CTAs); partials and the combine pass must give the same rows as whole tiles."""
    w = W.custom_workload([16000, 16100, 15900, 16200], [64, 64, 64, 64], 4, 2, 128, 64, seed=31, spare_pages=4)
    res, _ = _full_parity(w, opts=wpp.PlanOpts(0, 0, 0, 6))
    info = res["plan"].info
    assert info.num_tiles == 6 + 2 * 3 and info.num_split_tiles == 6 and info.workspace_bytes > 256


def test_a_wave_captured_in_a_cuda_graph_replays_bit_identically():
    """Both calls only enqueue work on the stream they are given (a memset node and kernels): a wave whose plan stays
    the same can be captured once and replayed, which for the smallest waves halves the time per wave."""
    w = W.cfg1()
    inp = cpu_inputs(w)
    _, _, ref, _ = run_oracle(w, inp)
    dev_inp = H.device_inputs(w, inp)
    c, d = H.ctx(), H.desc_of(w)
    plan = wpp.wpp_plan_tiles(c, d, w.prefix_lens, w.chunk_lens).to_device()
    dev = torch.device("cuda")
    bt = torch.from_numpy(w.block_tables).to(dev)
    P = torch.from_numpy(np.asarray(w.prefix_lens, dtype=np.int32)).to(dev)
    C = torch.from_numpy(np.asarray(w.chunk_lens, dtype=np.int32)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = torch.empty(w.total_new_tokens, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(max(256, int(plan.info.workspace_bytes)), dtype=torch.uint8, device=dev)

    def wave():
        wpp.wpp_kv_append(c, d, dev_inp["k_new"], dev_inp["v_new"], dev_inp["k_pool"], dev_inp["v_pool"], bt, P, C, plan,
                          status=status)
        wpp.wpp_prefill_attention_varlen(c, d, dev_inp["q"], out, None, dev_inp["k_pool"], dev_inp["v_pool"], bt, P, C,
                                         plan, workspace=ws, status=status)

    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        wave()                                           # first call outside the capture (one-time function attributes)
        s.synchronize()
        direct = out.clone()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            wave()
        for _ in range(3):
            out.view(torch.int16).fill_(0x7FC0)
            g.replay()
            s.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(out.view(torch.int16), direct.view(torch.int16))
    H.assert_close(f64(out), ref, "replayed wave")


def test_rescale_before_and_after_the_exponentials_and_the_library_choosing():
    """Scores that keep growing along the sequence (K scaled by 2^floor(pos / 4096)) move the row references on most
    key steps.  Both orders of work stay within the tolerance; with the choice left to the library it goes to
    "after" once its kernels have counted enough such steps, and back once a wave without them has run."""
    c = H.ctx()
    grow = W.custom_workload([45056], [256], 2, 1, 128, 64, seed=41, spare_pages=4, k_scale="cumulative")
    calm = W.custom_workload([45056], [256], 2, 1, 128, 64, seed=42, spare_pages=4)
    inp_g, inp_c = cpu_inputs(grow), cpu_inputs(calm)
    _, _, ref_g, _ = run_oracle(grow, inp_g)
    _, _, ref_c, _ = run_oracle(calm, inp_c)
    opts = wpp.PlanOpts(256, 0, 1, 0, 0, 1)              # whole 256-row tiles on the SM-wide kernel
    try:
        for mode in (0, 1):
            c.set_rescale_mode(mode)
            for w, inp, ref in ((grow, inp_g, ref_g), (calm, inp_c, ref_c)):
                res = H.run_wave(w, H.device_inputs(w, inp), opts=opts)
                assert res["status"] == 0
                H.assert_close(f64(res["out"]), ref, f"{w.name} rescale mode {mode}")
        c.set_rescale_mode(2)
        s0, m0, _ = c.rescale_stats()
        for _ in range(2):                               # per wave: 2 tiles x 4 warps x (353 + 354) key steps of the halves
            res = H.run_wave(grow, H.device_inputs(grow, inp_g), opts=opts)
            H.assert_close(f64(res["out"]), ref_g, "growing scores, library's choice")
        s1, m1, late = c.rescale_stats()
        assert s1 - s0 == 2 * 2 * 4 * (353 + 354) and (m1 - m0) * 10 >= (s1 - s0) * 3 and late
        for _ in range(2):
            res = H.run_wave(calm, H.device_inputs(calm, inp_c), opts=opts)
            H.assert_close(f64(res["out"]), ref_c, "calm scores, library's choice")
        s2, m2, late = c.rescale_stats()
        assert (m2 - m1) * 20 < (s2 - s1) * 3 and not late
    finally:
        c.set_rescale_mode(0)


def test_explicit_scale():
    w = W.custom_workload([70], [150], 2, 1, 128, 64, seed=10)
    _full_parity(w, sm_scale=0.05)


def test_empty_wave_is_a_no_op():
    w = W.custom_workload([10, 20], [0, 0], 2, 1, 64, 16, seed=11)
    res = H.run_wave(w, H.device_inputs(w))
    assert res["status"] == 0 and res["out"].numel() == 0


@pytest.mark.parametrize("shape", [1, 2])
def test_results_are_bit_reproducible(shape):
    w = W.custom_workload([500, 77], [260, 300], 8, 2, 128, 64, seed=12)
    inp = cpu_inputs(w)
    a = H.run_wave(w, H.device_inputs(w, inp), opts=wpp.PlanOpts(256, 0, 3, 0), shape=shape)
    b = H.run_wave(w, H.device_inputs(w, inp), opts=wpp.PlanOpts(256, 0, 3, 0), shape=shape)
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))
    assert torch.equal(a["lse"], b["lse"])


@pytest.mark.parametrize("shape", [1, 2])
def test_results_do_not_depend_on_which_cta_takes_which_tile(shape):
    """Tiles are handed out at run time, so the assignment differs from run to run and with the order option; the
    tiles themselves (and the fixed combine order) are the same, so every bit of the result must be too."""
    w = W.custom_workload([1500, 40, 900, 0, 2048, 300], [700, 512, 130, 260, 64, 333], 8, 2, 128, 64, seed=21)
    inp = cpu_inputs(w)
    ref = None
    for order in (0, 1, 0, 1):
        for splits in (1, 3):
            r = H.run_wave(w, H.device_inputs(w, inp), opts=wpp.PlanOpts(256, 0, splits, 0, order), shape=shape)
            assert r["status"] == 0
            key = (splits,)
            ref = ref or {}
            if key not in ref:
                ref[key] = (r["out"].view(torch.int16).clone(), r["lse"].clone())
            else:
                assert torch.equal(ref[key][0], r["out"].view(torch.int16)), (order, splits)
                assert torch.equal(ref[key][1], r["lse"]), (order, splits)


def test_stale_slots_unused_pages_and_scratch_poison_do_not_matter():
    """NaN bit patterns everywhere the method must not look: slots past the sequence end, unreferenced pages."""
    w = W.custom_workload([90, 3, 0], [40, 200, 5], 4, 2, 128, 64, seed=13, spare_pages=6)
    inp = cpu_inputs(w)
    kp, vp = bits(inp["k_pool"]).copy(), bits(inp["v_pool"]).copy()
    live = np.zeros((w.num_pages, w.page_size), dtype=bool)
    for i in range(w.num_requests):
        for pos in range(int(w.prefix_lens[i])):
            live[w.block_tables[i, pos // w.page_size], pos % w.page_size] = True
    dead = np.broadcast_to(~live[:, None, :, None], kp.shape)
    kp[dead] = 0x7FC0
    vp[dead] = 0xFFFF
    inp = dict(inp, k_pool=from_bits(kp), v_pool=from_bits(vp))
    _full_parity(w, inp=inp)
    _full_parity(w, inp=inp, opts=wpp.PlanOpts(0, 0, 2, 0))


@pytest.mark.parametrize("shape", [1, 2])
def test_page_permutation_gives_identical_bits(shape):
    w = W.custom_workload([200, 0], [130, 260], 4, 2, 128, 64, seed=14, spare_pages=4)
    inp = cpu_inputs(w)
    a = H.run_wave(w, H.device_inputs(w, inp), shape=shape)
    perm = np.random.default_rng(15).permutation(w.num_pages)
    kp = torch.empty_like(inp["k_pool"]); vp = torch.empty_like(inp["v_pool"])
    kp[perm] = inp["k_pool"]; vp[perm] = inp["v_pool"]
    w2 = W.custom_workload([200, 0], [130, 260], 4, 2, 128, 64, seed=14, spare_pages=4)
    w2.block_tables = np.where(w.block_tables >= 0, perm[np.maximum(w.block_tables, 0)], -1).astype(np.int32)
    b = H.run_wave(w2, H.device_inputs(w2, dict(inp, k_pool=kp, v_pool=vp)), shape=shape)
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))


def test_successive_chunks_on_one_stream_equal_one_shot():
    """Chunks of one request in successive calls (order kept by the stream) give the rows of one call."""
    n, Hq, Hkv, d, B = 700, 4, 2, 128, 64
    w_all = W.custom_workload([0], [n], Hq, Hkv, d, B, seed=16)
    inp = cpu_inputs(w_all)
    _, _, ref, _ = run_oracle(w_all, inp)
    dev = H.device_inputs(w_all, inp)
    outs, start = [], 0
    for c in (130, 1, 300, 269):
        w = W.custom_workload([start], [c], Hq, Hkv, d, B, seed=16)
        w.block_tables = np.full((1, w_all.max_blocks_per_req), -1, dtype=np.int32)
        w.block_tables[0, :] = w_all.block_tables[0]
        w.num_pages = w_all.num_pages
        part = dict(q=dev["q"][start:start + c], k_new=dev["k_new"][start:start + c],
                    v_new=dev["v_new"][start:start + c], k_pool=dev["k_pool"], v_pool=dev["v_pool"])
        res = H.run_wave(w, part)
        assert res["status"] == 0
        outs.append(f64(res["out"]))
        start += c
    H.assert_close(np.concatenate(outs), ref, "successive chunks")


def test_a_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """Every device-side wait is bounded: a barrier nothing arrives on makes the wait give up after its limit,
    the kernel ends normally and the status word says WPP_ERR_TIMEOUT (no hang, no trap)."""
    c = H.ctx()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    limit = 2_000_000                                    # about a millisecond of SM clocks
    wpp.wpp_selftest_bounded_wait(c, limit, status, waited)
    torch.cuda.synchronize()
    assert int(status.item()) == 8                       # WPP_ERR_TIMEOUT
    assert limit < int(waited.item()) < 50 * limit
    _full_parity(W.custom_workload([64], [64], 2, 1, 128, 64, seed=17))      # the context still works


@pytest.mark.parametrize("shape", [1, 2])
def test_bad_page_id_sets_status_without_trapping(shape):
    w = W.custom_workload([64], [64], 2, 1, 128, 64, seed=17)
    w.block_tables = w.block_tables.copy()
    w.block_tables[0, 1] = w.num_pages + 5
    res = H.run_wave(w, H.device_inputs(w), shape=shape)
    assert res["status"] == 3          # WPP_ERR_BOUNDS
    # the context is still usable
    w2 = W.custom_workload([64], [64], 2, 1, 128, 64, seed=17)
    _full_parity(w2)


@pytest.mark.parametrize("shape", [1, 2])
@pytest.mark.parametrize("splits", [1, 2])
def test_plan_launched_with_other_lengths_is_refused_per_request(splits, shape):
    """Section 4.6: a position mismatch fails execution instead of running against the wrong cache state.  The
    plan is made for one set of spans; the device arrays are altered afterwards (on the host): the requests
    whose span differs are refused - status WPP_ERR_PLAN_MISMATCH, none of their slots written, none of their
    rows computed - the others run normally, nothing traps and the context stays usable."""
    w = W.custom_workload([200, 128, 0, 300], [150, 260, 70, 129], 4, 2, 128, 64, seed=29, spare_pages=4)
    inp = cpu_inputs(w)
    P_dev = w.prefix_lens.copy()
    C_dev = w.chunk_lens.copy()
    P_dev[1] += 64          # this rank's cache of request 1 ends elsewhere
    C_dev[3] -= 1           # request 3's span has another length
    res = H.run_wave(w, H.device_inputs(w, inp), opts=wpp.PlanOpts(0, 0, splits, 0), launch_prefix_lens=P_dev,
                     launch_chunk_lens=C_dev, shape=shape)
    assert res["status"] == 6                                    # WPP_ERR_PLAN_MISMATCH
    # the oracle's wave without the refused requests: their chunks are empty
    C_ok = w.chunk_lens.copy()
    C_ok[[1, 3]] = 0
    off = w.q_offsets
    keep = np.concatenate([np.arange(off[i], off[i + 1]) for i in (0, 2)])
    kp, vp = oracle.oracle_append(inp["k_new"][keep], inp["v_new"][keep], inp["k_pool"], inp["v_pool"],
                                  w.block_tables, w.prefix_lens, C_ok)
    assert np.array_equal(bits(res["k_pool"]), kp), "a refused request's slots were written"
    assert np.array_equal(bits(res["v_pool"]), vp)
    ref, ref_lse = oracle.oracle_attention(inp["q"][keep], kp, vp, w.block_tables, w.prefix_lens, C_ok)
    H.assert_close(f64(res["out"][keep]), ref, "requests whose spans agree")
    for i in (1, 3):
        rows = res["out"][off[i]:off[i + 1]].float()
        # unsplit tiles leave the rows as the caller's poison; split tiles read as zero after the combine
        assert bool((torch.isnan(rows) | (rows == 0)).all()), "a refused request's rows were computed"
    _full_parity(W.custom_workload([64], [64], 2, 1, 128, 64, seed=17))      # the context still works


def test_cfg2_sampled_rows():
    """Ragged batch of 16: the oracle checks a seeded sample of (request, row, head) plus boundary rows."""
    w = W.cfg2()
    inp = cpu_inputs(w)
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"], w.block_tables,
                                  w.prefix_lens, w.chunk_lens)
    res = H.run_wave(w, H.device_inputs(w, inp))
    assert res["status"] == 0
    assert np.array_equal(bits(res["k_pool"]), kp) and np.array_equal(bits(res["v_pool"]), vp)
    rng = np.random.default_rng(202)
    units = []
    for i in range(w.num_requests):
        C = int(w.chunk_lens[i])
        for t in sorted({0, 1, 63, 64, 127, 128, C // 2, C - 2, C - 1}):
            if 0 <= t < C:
                units += [(i, t, h) for h in (0, 7, 31)]
    for _ in range(600):
        i = int(rng.integers(w.num_requests))
        units.append((i, int(rng.integers(w.chunk_lens[i])), int(rng.integers(w.num_q_heads))))
    units = np.array(units, dtype=np.int32)
    ref, ref_lse = oracle.oracle_attention_units(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, units)
    off = w.q_offsets
    rows = torch.from_numpy(off[units[:, 0]] + units[:, 1]).cuda()
    heads = torch.from_numpy(units[:, 2].astype(np.int64)).cuda()
    got = f64(res["out"][rows, heads])
    print("cfg2", H.assert_close(got, ref, "cfg2 sample"))
    got_lse = res["lse"][rows, heads].double().cpu().numpy()
    assert np.abs(got_lse - ref_lse).max() < 2e-2
    assert not torch.isnan(res["out"].float()).any()
