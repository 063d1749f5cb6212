"""Host logic of the C-ABI library (no GPU): symbol exports, argument checks, and the work split.

The plan is checked by brute force on small waves: every visible (request, row, head, key) pair is covered
exactly once, no tile lies wholly above the diagonal, split parts tile a tile's key range contiguously, every
tile is owned by exactly one persistent CTA, and equal inputs give byte-identical plans.
"""
import ctypes
import os
import re
import struct

import numpy as np
import pytest

import paper_2609_35263_b200 as wpp
from paper_2609_35263_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HDR_FMT = "<IIQ" + "i" * 8 + "qqq" + "QQ" + "IIII" + "ii"      # WppPlanHeader up to the kernel shape


def parse_plan(plan):
    raw = plan.host_bytes()
    f = struct.unpack_from(HDR_FMT, raw, 0)
    (magic, version, desc_hash, R, num_ctas, num_units, num_combine, num_slots, tile_m, tile_n, head_dim,
     T, key_steps, flops, ws_bytes, plan_bytes, off_q, off_prefix, off_units, off_comb, shape, nonempty_halves) = f
    assert magic == 0x31505057
    q_off = np.frombuffer(raw, dtype=np.int32, count=R + 1, offset=off_q)
    units = np.frombuffer(raw, dtype=np.int32, count=num_units * 12, offset=off_units).reshape(num_units, 12)
    comb = np.frombuffer(raw, dtype=np.int32, count=num_combine * 8, offset=off_comb).reshape(num_combine, 8)
    keys = ["request", "kv_begin", "kv_end", "split_slot", "row0_a", "row0_b", "rows_a", "rows_b", "head_a",
            "head_b", "cost", "pack"]
    prefix = np.frombuffer(raw, dtype=np.int32, count=R, offset=off_prefix)
    return dict(R=R, num_ctas=num_ctas, tile_m=tile_m, T=T, key_steps=key_steps, flops=flops, slots=num_slots,
                ws_bytes=ws_bytes, q_off=q_off, comb=comb, shape=shape, nonempty_halves=nonempty_halves, prefix=prefix,
                units=[dict(zip(keys, u.tolist())) for u in units])


def desc(R, Hq, Hkv, d, B, max_blocks, pages=1000):
    return wpp.make_desc(R, Hq, Hkv, d, B, max_blocks, pages)


def test_library_exports_every_declared_symbol():
    lib = wpp.load_library()
    hdr = open(os.path.join(ROOT, "include", "wpp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)            # declarations only, not the prose
    declared = set(re.findall(r"\b(wpp_[a-z_0-9]+)\s*\(", hdr))
    assert {"wpp_plan_tiles", "wpp_kv_append", "wpp_prefill_attention_varlen"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in wpp.h but not exported"
    assert set(binding.EXPORTS) <= declared


def test_status_strings():
    lib = wpp.load_library()
    assert lib.wpp_status_string(0) == b"WPP_OK"
    assert lib.wpp_status_string(4) == b"WPP_ERR_POSITION_MISMATCH"


@pytest.mark.parametrize("P,C,Hq,Hkv,tile_m,splits", [
    ([0], [1], 2, 1, 0, 0),
    ([37, 0, 300], [200, 129, 3], 4, 2, 128, 0),
    ([37, 0, 300], [200, 129, 3], 4, 2, 256, 0),
    ([1000, 5], [700, 300], 4, 2, 256, 3),
    ([1000, 5], [700, 300], 3, 1, 256, 2),          # odd group: unpaired tails
    ([0, 0, 0], [64, 0, 128], 8, 2, 256, 7),
    ([130], [64], 4, 2, 256, 2),
    ([300, 5, 0], [16, 33, 7], 16, 2, 256, 2),      # short chunks: 8, 2 and 8 heads packed per half
    ([300, 5], [16, 64], 8, 1, 128, 0),
])
def test_plan_covers_every_visible_pair_exactly_once(P, C, Hq, Hkv, tile_m, splits):
    B = 16
    mb = max(1, max((p + c + B - 1) // B for p, c in zip(P, C)))
    d = desc(len(P), Hq, Hkv, 128, B, mb)
    plan = wpp.wpp_plan_tiles(None, d, P, C, opts=wpp.PlanOpts(tile_m, 0, splits, 40), pin=False)
    pl = parse_plan(plan)
    assert pl["T"] == sum(C) and pl["q_off"].tolist() == np.concatenate([[0], np.cumsum(C)]).tolist()
    assert pl["shape"] in (1, 2) and 1 <= pl["num_ctas"] <= 40 * pl["shape"]     # the small shape runs two CTAs per SM
    assert pl["prefix"].tolist() == list(P)                                      # the spans the kernels check against
    assert pl["nonempty_halves"] == sum((u["rows_a"] > 0) + (u["rows_b"] > 0) for u in pl["units"])
    G = Hq // Hkv
    cover = {}
    steps_total = 0
    for u in pl["units"]:
        i = u["request"]
        assert u["kv_begin"] < u["kv_end"]
        any_work = False
        for hf in "ab":
            rows, row0, head = u["rows_" + hf], u["row0_" + hf], u["head_" + hf]
            if rows == 0:
                continue
            pack = u["pack"]
            assert pack in (1, 2, 4, 8) and 0 < rows <= 128 // pack and row0 + rows <= C[i]
            assert 0 <= head and head + pack <= Hq
            assert head // G == (head + pack - 1) // G == u["head_a"] // G      # one KV head per tile
            end = (P[i] + row0 + rows + 127) // 128
            n = max(0, min(u["kv_end"], end) - u["kv_begin"])
            steps_total += n
            any_work |= n > 0
            for hd_ in range(head, head + pack):
                for t in range(row0, row0 + rows):
                    last = P[i] + t                              # last visible key
                    lo, hi = u["kv_begin"] * 128, min(u["kv_end"], end) * 128
                    for key in range(lo, min(hi, last + 1)):
                        k = (i, t, hd_, key)
                        cover[k] = cover.get(k, 0) + 1
        assert any_work, "a tile with nothing to compute"
    assert steps_total == pl["key_steps"]
    want = sum(Hq * (c * p + c * (c + 1) // 2) for p, c in zip(P, C))
    assert len(cover) == want and all(v == 1 for v in cover.values())
    assert pl["flops"] == 4 * 128 * want
    # split parts of a half tile use consecutive slots and contiguous key ranges starting at 0
    by_slot = {u["split_slot"]: u for u in pl["units"] if u["split_slot"] >= 0}
    assert len(by_slot) == pl["slots"]
    for c in pl["comb"]:
        req, row0, rows, head, slot0, ns, half, lane0 = c.tolist()
        parts = [by_slot[s] for s in range(slot0, slot0 + ns)]
        assert parts[0]["kv_begin"] == 0 and all(a["kv_end"] == b["kv_begin"] for a, b in zip(parts, parts[1:]))
        hf = "ab"[half]
        assert all(p_["request"] == req and p_["row0_" + hf] == row0 and p_["rows_" + hf] == rows and
                   p_["head_" + hf] + lane0 // (128 // p_["pack"]) == head and lane0 % (128 // p_["pack"]) == 0
                   for p_ in parts)
        assert parts[-1]["kv_end"] >= (P[req] + row0 + rows + 127) // 128
    if splits >= 2 and max((p + c + 127) // 128 for p, c in zip(P, C)) >= 2:
        assert pl["slots"] > 0 and pl["ws_bytes"] >= 256 + pl["slots"] * 2 * 128 * 129 * 4


def _greedy_finish_times(costs, n_ctas):
    """Finish time of every CTA when free CTAs take the tiles in list order (what the kernel's counter does)."""
    import heapq
    heap = [(0, c) for c in range(n_ctas)]
    for cost in costs:
        t, c = heapq.heappop(heap)
        heapq.heappush(heap, (t + max(1, cost), c))
    return [t for t, _ in heap]


def test_plan_is_deterministic_and_its_order_balances():
    rng = np.random.default_rng(5)
    P = (rng.integers(0, 100, 24) * 64).tolist()
    C = rng.integers(1, 2000, 24).tolist()
    d = desc(24, 16, 4, 128, 64, 200)
    for order in (0, 1):
        opts = wpp.PlanOpts(0, 0, 0, 0, order, 1)
        a = wpp.wpp_plan_tiles(None, d, P, C, opts=opts, pin=False)
        b = wpp.wpp_plan_tiles(None, d, P, C, opts=opts, pin=False)
        assert a.host_bytes() == b.host_bytes()
        pl = parse_plan(a)
        costs = [u["cost"] for u in pl["units"]]
        finish = _greedy_finish_times(costs, pl["num_ctas"])
        assert max(finish) - min(finish) <= max(costs)     # taking tiles in order: nobody idles longer than one tile
        if order == 1:                                     # longest first
            assert costs == sorted(costs, reverse=True)
        else:                                              # stream order: KV head major, a request's tiles together
            kv = [u["head_a"] // 4 for u in pl["units"]]
            assert kv == sorted(kv)
            for g in range(4):
                reqs = [u["request"] for u in pl["units"] if u["head_a"] // 4 == g]
                runs = [r for i, r in enumerate(reqs) if i == 0 or reqs[i - 1] != r]
                assert len(runs) == len(set(runs))         # each request appears as one contiguous run


def test_stream_order_runs_the_tiles_of_one_kv_stream_together():
    d = desc(3, 16, 4, 128, 64, 200)
    pl = parse_plan(wpp.wpp_plan_tiles(None, d, [4096, 0, 8192], [1024, 512, 256], opts=wpp.PlanOpts(256, 0, 1, 8, 0, 1),
                                       pin=False))
    # the first tiles (one per CTA) belong to KV head 0 of the costliest request (request 0: 4 row blocks x 4 heads)
    firsts = pl["units"][:pl["num_ctas"]]
    assert all(u["request"] == 0 and u["head_a"] // 4 == 0 for u in firsts)


def test_short_row_blocks_pack_heads_of_one_kv_group():
    d = desc(1, 8, 2, 128, 64, 10)                  # G = 4
    pl = parse_plan(wpp.wpp_plan_tiles(None, d, [0], [300], opts=wpp.PlanOpts(256, 0, 1, 148), pin=False))
    tails = [u for u in pl["units"] if u["row0_a"] == 256]          # 44 rows: two heads per half, four per tile
    assert len(tails) == 2 and all(u["pack"] == 2 and u["rows_a"] == 44 and u["rows_b"] == 44 and
                                   u["row0_b"] == 256 and u["head_b"] == u["head_a"] + 2 for u in tails)
    full = [u for u in pl["units"] if u["row0_a"] == 0]
    assert len(full) == 8 and all(u["pack"] == 1 and u["rows_b"] == 128 and u["row0_b"] == 128 for u in full)
    d8 = desc(1, 16, 2, 128, 64, 10)                # G = 8, a 10-row chunk: all 8 heads of a group in one half
    pl8 = parse_plan(wpp.wpp_plan_tiles(None, d8, [70], [10], opts=wpp.PlanOpts(256, 0, 1, 148), pin=False))
    assert [(u["pack"], u["head_a"], u["rows_b"]) for u in pl8["units"]] == [(8, 0, 0), (8, 8, 0)]
    d100 = desc(1, 8, 2, 128, 64, 10)               # 100 rows do not fit twice into 128: one head per half
    pl100 = parse_plan(wpp.wpp_plan_tiles(None, d100, [0], [100], opts=wpp.PlanOpts(256, 0, 1, 148), pin=False))
    assert all(u["pack"] == 1 and u["head_b"] == u["head_a"] + 1 for u in pl100["units"]) and len(pl100["units"]) == 4


def test_few_tiles_fall_back_to_128_row_tiles_and_split_keys():
    d = desc(1, 8, 2, 64, 16, 64)
    pl = parse_plan(wpp.wpp_plan_tiles(None, d, [256], [128], pin=False))       # the single-request configuration
    assert pl["tile_m"] == 128 and len(pl["units"]) == 8 and all(u["rows_b"] == 0 for u in pl["units"])
    d2 = desc(1, 2, 1, 128, 64, 600)
    pl2 = parse_plan(wpp.wpp_plan_tiles(None, d2, [32768], [128], pin=False))
    assert pl2["slots"] > 0 and len(pl2["units"]) > 100                          # long prefix, two tiles: split along keys


def test_a_partly_filled_last_round_of_long_tiles_is_cut_along_the_keys():
    """32 requests of 64 new tokens over a 32,768-token prefix, 64/8 heads: 512 tiles of 257 key steps per half on 148
    CTAs are three full rounds and 68 tiles; those 68 are cut in two so that the last round takes half a tile's time.
    Nothing is cut when the rounds divide evenly, when the tiles are short, or when the caller says 1 (never)."""
    R, P, C = 32, 32768, 64
    d = desc(R, 64, 8, 128, 64, 520, pages=20000)
    pl = parse_plan(wpp.wpp_plan_tiles(None, d, [P] * R, [C] * R, opts=wpp.PlanOpts(0, 0, 0, 148), pin=False))
    units = pl["units"]
    whole = [u for u in units if u["split_slot"] < 0]
    cut = [u for u in units if u["split_slot"] >= 0]
    assert len(whole) == 512 - 68 and len(cut) == 2 * 68 and pl["slots"] == 2 * 68
    assert all(u["split_slot"] >= 0 for u in units[len(whole):])              # the cut tiles are the last in the order
    assert sorted(u["kv_end"] - u["kv_begin"] for u in cut[:2]) == [128, 129] and cut[0]["kv_end"] == cut[1]["kv_begin"]
    assert sum(u["cost"] for u in units) == pl["key_steps"] == 512 * 2 * 257
    finish = _greedy_finish_times([u["cost"] + 3 for u in units], 148)
    assert max(finish) <= 3.6 * (514 + 3)                                      # against 4 rounds uncut
    never = parse_plan(wpp.wpp_plan_tiles(None, d, [P] * R, [C] * R, opts=wpp.PlanOpts(0, 0, 1, 148), pin=False))
    assert never["slots"] == 0 and len(never["units"]) == 512
    even = parse_plan(wpp.wpp_plan_tiles(None, d, [P] * R, [C] * R, opts=wpp.PlanOpts(0, 0, 0, 128), pin=False))
    assert even["slots"] == 0                                                  # 512 tiles on 128 CTAs: four full rounds
    short = parse_plan(wpp.wpp_plan_tiles(None, d, [4096] * R, [C] * R, opts=wpp.PlanOpts(0, 0, 0, 148), pin=False))
    assert short["slots"] == 0                                                 # 33 key steps per half: not worth a cut


def _status(fn, *a, **k):
    try:
        fn(*a, **k)
        return 0
    except wpp.WppError as e:
        return e.status


def test_host_detectable_errors_are_reported_before_any_launch():
    ok = desc(2, 4, 2, 128, 64, 4)
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, 64], [100, 64], pin=False) == 0
    # table too short for P + C
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, 200], [100, 64], pin=False) == 3
    # span start differs from what the cache holds: execution must fail, not run against the wrong state
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, 64], [100, 64], cached_lens=[0, 128], pin=False) == 4
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, 64], [100, 64], cached_lens=[0, 64], pin=False) == 0
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, -1], [100, 64], pin=False) == 1
    assert _status(wpp.wpp_plan_tiles, None, desc(1, 4, 2, 96, 64, 4), [0], [1], pin=False) == 2     # head_dim
    assert _status(wpp.wpp_plan_tiles, None, desc(1, 4, 2, 128, 48, 4), [0], [1], pin=False) == 2    # page size
    assert _status(wpp.wpp_plan_tiles, None, desc(1, 5, 2, 128, 64, 4), [0], [1], pin=False) == 2    # head ratio
    bad_stride = wpp.make_desc(1, 4, 2, 128, 64, 4, 10, q_head_stride=132)
    assert _status(wpp.wpp_plan_tiles, None, bad_stride, [0], [1], pin=False) == 1
    assert _status(wpp.wpp_plan_tiles, None, ok, [0, 0], [1, 1], opts=wpp.PlanOpts(64, 0, 0, 0), pin=False) == 2


def test_validate_batch_finds_aliased_appends():
    d = desc(2, 2, 1, 128, 16, 4, pages=8)
    bt = np.array([[0, 1, -1, -1], [2, 3, -1, -1]], dtype=np.int32)
    assert wpp.wpp_validate_batch(d, bt, [10, 0], [10, 20]) == 0
    bt2 = bt.copy(); bt2[1, 1] = 1                                   # both requests write page 1
    assert wpp.wpp_validate_batch(d, bt2, [10, 0], [10, 20]) == 9
    bt3 = bt.copy(); bt3[1, 0] = 0                                   # request 1 writes what request 0 reads
    assert wpp.wpp_validate_batch(d, bt3, [10, 0], [10, 5]) == 9
    shared = np.array([[0, 1, -1, -1], [0, 2, -1, -1]], dtype=np.int32)   # a shared, read-only prefix page is fine
    assert wpp.wpp_validate_batch(d, shared, [16, 16], [4, 4]) == 0
    bt4 = bt.copy(); bt4[0, 1] = 8
    assert wpp.wpp_validate_batch(d, bt4, [10, 0], [10, 20]) == 3
    assert wpp.wpp_validate_batch(d, bt, [10, 0], [100, 20]) == 3


def test_there_is_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(wpp.WppError):
        wpp.Context(0)


def test_kernel_shape_follows_the_mean_key_steps_per_half():
    """Short tiles go to the small kernel shape (two CTAs per SM), long ones to the SM-wide one; an explicit choice
    is kept; the shape is part of the plan."""
    d = desc(4, 8, 2, 128, 64, 300)
    short = wpp.wpp_plan_tiles(None, d, [0, 0, 0, 0], [64, 100, 64, 128], pin=False)
    long_ = wpp.wpp_plan_tiles(None, d, [16000, 9000, 12000, 8000], [256, 300, 64, 500], pin=False)
    assert short.info.shape == 2 and parse_plan(short)["shape"] == 2
    assert long_.info.shape == 1 and parse_plan(long_)["shape"] == 1
    assert short.info.num_ctas == min(2 * 148, 2 * short.info.num_tiles)
    for shape in (1, 2):
        forced = wpp.wpp_plan_tiles(None, d, [0, 64, 0, 128], [256, 300, 64, 500], opts=wpp.PlanOpts(0, 0, 0, 0, 0, shape),
                                    pin=False)
        assert forced.info.shape == shape
    with pytest.raises(wpp.WppError):
        wpp.wpp_plan_tiles(None, d, [0] * 4, [64] * 4, opts=wpp.PlanOpts(0, 0, 0, 0, 0, 3), pin=False)
