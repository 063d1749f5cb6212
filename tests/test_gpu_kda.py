"""wpp_kda_chunk (CUDA, through the C ABI) against the fp64 oracle of the recurrent-state layer (Section 3.1 update,
Section 3.2 snapshots), element by element on seeded inputs, plus the properties that hold at any size.

Tolerances: the token-by-token forms (layouts 1, 2) compute in fp32 (relative error of a step about 1e-7, a few
1e-6 after thousands of contracting steps); the chunk-parallel tensor-core form (layout 3) multiplies operands of
16 significant bits (two bf16 terms each, relative 2^-17 per factor) and accumulates in fp32, so a product of 64 or
128 terms carries about 1e-5 of its typical term; all forms round outputs to bf16 (relative 2^-9), states stay fp32.
  outputs : |delta| <= 2^-8 |ref| + 1e-4 max|ref|          states : |delta| <= 1e-4 max|ref|"""
import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from oracle import kda as O
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


def _oracle(w, t, heads=None):
    hs = slice(None) if heads is None else heads
    f = lambda x: x[:, hs].double().numpy()
    pool = t["state_pool"][:, hs].double().numpy().copy()
    o = O.kda_chunk(f(t["q"]), f(t["k"]), f(t["v"]), f(t["alpha"]), f(t["beta"]), w.chunk_lens, pool, w.state_in,
                    w.state_out, w.prefix_lens, w.snap_interval, w.snap_slots)
    return o, pool


def _gpu(w, t, state_in=None, state_out=None, layout=0):
    dev = torch.device("cuda")
    d = {k: v.to(dev) for k, v in t.items()}
    i32 = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    T, Hh = int(t["q"].shape[0]), int(t["q"].shape[1])
    ws = torch.full((wpp.wpp_kda_workspace_bytes(len(w.chunk_lens), Hh, T),), 0xFF, dtype=torch.uint8, device=dev)
    out = wpp.wpp_kda_chunk(H.ctx(), d["q"], d["k"], d["v"], d["alpha"], d["beta"],
                            torch.from_numpy(w.row_offsets).to(dev), d["state_pool"],
                            i32(w.state_in if state_in is None else state_in),
                            i32(w.state_out if state_out is None else state_out),
                            prefix_lens=i32(w.prefix_lens), snap_interval=w.snap_interval,
                            snap_slots=i32(w.snap_slots), status=status, layout=layout, workspace=ws)
    torch.cuda.synchronize()
    return out.float().cpu().double().numpy(), d["state_pool"].cpu().double().numpy(), int(status.item())


def _close_out(got, ref, what):
    if ref.size == 0:
        return
    bound = 2.0 ** -8 * np.abs(ref) + 1e-4 * np.abs(ref).max()
    bad = np.abs(got - ref) > bound
    assert not bad.any(), f"{what}: {bad.sum()} outputs off, worst {np.abs(got - ref).max():.3e}"


def _close_state(got, ref, what):
    assert np.abs(got - ref).max() <= 1e-4 * max(np.abs(ref).max(), 1e-30), f"{what}: {np.abs(got - ref).max():.3e}"


@pytest.mark.parametrize("lens,prefix,interval,H_", [
    ([37, 5, 64, 0, 1, 16, 17, 130], [11, 0, 128, 7, 0, 16, 3, 1000], 16, 2),     # ragged, stage tails, empty chunk
    ([300], [0], 0, 3),                                                            # one request from the zero state
    ([15, 16, 17, 31, 32, 33], [1, 2, 3, 4, 5, 6], 7, 1),                          # around the staging size; odd interval
])
@pytest.mark.parametrize("layout", [1, 2, 3])       # one CTA per (request, head) / four column slices / chunk-parallel
def test_ragged_batches_match_the_oracle(lens, prefix, interval, H_, layout):
    w = W.kda_workload("ragged", 11, lens, H_, prefix, snap_interval=interval)
    t = w.tensors()
    ref_o, ref_pool = _oracle(w, t)
    got_o, got_pool, status = _gpu(w, t, layout=layout)
    assert status == 0
    _close_out(got_o, ref_o, "outputs")
    _close_state(got_pool, ref_pool, "state pool")
    # slots nobody writes keep their bits
    written = set(int(s) for s in w.state_out if s >= 0)
    if w.snap_slots is not None:
        written |= set(int(s) for s in w.snap_slots.ravel() if s >= 0)
    for s in range(w.num_slots):
        if s not in written:
            assert np.array_equal(got_pool[s], t["state_pool"][s].double().numpy())


@pytest.mark.parametrize("layout", [1, 2, 3])
def test_a_long_chain_stays_within_tolerance(layout):
    w = W.kda_workload("long", 5, [2048], 1, [4096])
    t = w.tensors()
    ref_o, ref_pool = _oracle(w, t)
    got_o, got_pool, status = _gpu(w, t, layout=layout)
    assert status == 0
    _close_out(got_o, ref_o, "outputs")
    _close_state(got_pool, ref_pool, "state pool")


@pytest.mark.parametrize("layout,cut", [(1, (64, 32)), (1, (37, 20)), (2, (64, 32)), (2, (37, 20)), (3, (59, 64))])
def test_splitting_a_chunk_and_resuming_is_bit_identical(layout, cut):
    """Section 3.2: the state after exactly r tokens is all a recurrent layer needs.  The token-by-token forms'
    arithmetic per token does not depend on where a chunk starts, so one call and two resumed calls agree to the bit
    for any cut; the chunk-parallel form works on blocks of 64 sequence positions, so it does for cuts at multiples
    of 64 (request 0 has 5 cached tokens: its cut after 59 tokens is position 64)."""
    w = W.kda_workload("whole", 3, [100, 64], 2, [5, 0], resume=[True, False])
    t = w.tensors()
    whole_o, whole_pool, _ = _gpu(w, t, layout=layout)
    rows = w.row_offsets
    parts_o = np.zeros_like(whole_o)
    pool = t["state_pool"].clone()
    for first in (True, False):
        lens = [cut[i] if first else int(w.chunk_lens[i]) - cut[i] for i in range(2)]
        sel = np.concatenate([np.arange(rows[i] + (0 if first else cut[i]), rows[i] + (cut[i] if first else w.chunk_lens[i]))
                              for i in range(2)])
        wp = W.kda_workload("part", 3, lens, 2, [5, 0] if first else [5 + cut[0], cut[1]])
        wp.num_slots = w.num_slots
        tp = {k: (v[sel].contiguous() if k != "state_pool" else pool) for k, v in t.items()}
        s_in = w.state_in if first else w.state_out          # the second call resumes from what the first stored
        o, new_pool, status = _gpu(wp, tp, state_in=s_in, state_out=w.state_out, layout=layout)
        assert status == 0
        parts_o[sel] = o
        pool = torch.from_numpy(new_pool).float()
    assert np.array_equal(parts_o, whole_o)
    assert np.array_equal(pool.double().numpy(), whole_pool)


def test_splitting_inside_a_block_stays_within_tolerance_in_the_chunk_parallel_form():
    """A cut that is not a multiple of 64 moves a block boundary of the chunk-parallel form: the two resumed calls
    then round differently from the single call, and both stay within the tolerances against the oracle."""
    w = W.kda_workload("whole", 3, [100, 64], 2, [5, 0], resume=[True, False])
    t = w.tensors()
    ref_o, ref_pool = _oracle(w, t)
    rows, cut = w.row_offsets, (37, 20)
    parts_o = np.zeros_like(ref_o)
    pool = t["state_pool"].clone()
    for first in (True, False):
        lens = [cut[i] if first else int(w.chunk_lens[i]) - cut[i] for i in range(2)]
        sel = np.concatenate([np.arange(rows[i] + (0 if first else cut[i]), rows[i] + (cut[i] if first else w.chunk_lens[i]))
                              for i in range(2)])
        wp = W.kda_workload("part", 3, lens, 2, [5, 0] if first else [5 + cut[0], cut[1]])
        wp.num_slots = w.num_slots
        tp = {k: (v[sel].contiguous() if k != "state_pool" else pool) for k, v in t.items()}
        o, new_pool, status = _gpu(wp, tp, state_in=w.state_in if first else w.state_out, state_out=w.state_out, layout=3)
        assert status == 0
        parts_o[sel] = o
        pool = torch.from_numpy(new_pool).float()
    _close_out(parts_o, ref_o, "outputs of the two resumed calls")
    for i in range(2):
        _close_state(pool[w.state_out[i]].double().numpy(), ref_pool[w.state_out[i]], "final state")


@pytest.mark.parametrize("layout", [1, 2, 3])
def test_tiny_and_zero_decays(layout):
    """Decays of exactly 0 (a channel forgets everything), of 1e-6 and 1e-20, and runs of small ones."""
    w = W.kda_workload("decays", 17, [90, 40], 2, [3, 0])
    t = w.tensors()
    rng = np.random.default_rng(17)
    a = t["alpha"].numpy()
    T = a.shape[0]
    for val, count in ((0.0, 40), (1e-6, 40), (1e-20, 20), (0.3, 2000)):
        idx = (rng.integers(0, T, count), rng.integers(0, 2, count), rng.integers(0, 128, count))
        a[idx] = val
    a[50:58, 0, 7] = 0.05                                      # eight small decays in a row on one channel
    a[0, :, :] = 0.0                                           # the first token forgets the resumed state entirely
    ref_o, ref_pool = _oracle(w, t)
    got_o, got_pool, status = _gpu(w, t, layout=layout)
    assert status == 0 and np.isfinite(got_o).all() and np.isfinite(got_pool).all()
    _close_out(got_o, ref_o, "outputs")
    _close_state(got_pool, ref_pool, "state pool")


@pytest.mark.parametrize("layout", [1, 2, 3])
def test_in_place_slots_and_pure_decay(layout):
    # state_out == state_in updates a slot in place; with beta = 0 and alpha = 1 the state must not change at all
    w = W.kda_workload("inplace", 9, [50, 20], 2, [10, 10])
    t = w.tensors()
    t["beta"].zero_()
    t["alpha"].fill_(1.0)
    got_o, got_pool, status = _gpu(w, t, state_out=w.state_in, layout=layout)
    assert status == 0
    assert np.array_equal(got_pool, t["state_pool"].double().numpy())
    ref = np.einsum("rhkv,rhk->rhv", t["state_pool"][[0] * 50 + [1] * 20].double().numpy(), t["q"].double().numpy())
    _close_out(got_o, ref, "o = S0^T q")


def test_bad_slot_ids_are_reported_and_skipped():
    w = W.kda_workload("bad", 2, [20, 20, 20], 1, [4, 4, 4])
    t = w.tensors()
    s_in, s_out = w.state_in.copy(), w.state_out.copy()
    s_in[1], s_out[2] = w.num_slots + 5, -7
    got_o, got_pool, status = _gpu(w, t, state_in=s_in, state_out=s_out)
    assert status == 3                                                 # WPP_ERR_BOUNDS
    w.state_in, w.state_out = np.where(s_in >= w.num_slots, -1, s_in), np.where(s_out < -1, -1, s_out)
    ref_o, ref_pool = _oracle(w, t)                                    # bad ids behave like -1
    _close_out(got_o, ref_o, "outputs")
    _close_state(got_pool, ref_pool, "state pool")


def test_argument_errors():
    dev = torch.device("cuda")
    z = lambda *s, dt=torch.bfloat16: torch.zeros(*s, dtype=dt, device=dev)
    ro = torch.tensor([0, 4], dtype=torch.int64, device=dev)
    slot = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = z(1, 1, 64, 64, dt=torch.float32)
    with pytest.raises(wpp.WppError) as e:                            # d_k = d_v = 64 is not built
        wpp.wpp_kda_chunk(H.ctx(), z(4, 1, 64), z(4, 1, 64), z(4, 1, 64), z(4, 1, 64, dt=torch.float32),
                          z(4, 1, dt=torch.float32), ro, pool, slot, slot)
    assert e.value.status == 2
    pool = z(1, 1, 128, 128, dt=torch.float32)
    with pytest.raises(wpp.WppError) as e:                            # no such layout
        wpp.wpp_kda_chunk(H.ctx(), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128, dt=torch.float32),
                          z(4, 1, dt=torch.float32), ro, pool, slot, slot, layout=4)
    assert e.value.status == 1
    with pytest.raises(wpp.WppError) as e:                            # the chunk-parallel form needs its workspace
        wpp.wpp_kda_chunk(H.ctx(), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128, dt=torch.float32),
                          z(4, 1, dt=torch.float32), ro, pool, slot, slot, layout=3)
    assert e.value.status == 5
    small = torch.empty(1024, dtype=torch.uint8, device=dev)
    with pytest.raises(wpp.WppError) as e:
        wpp.wpp_kda_chunk(H.ctx(), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128, dt=torch.float32),
                          z(4, 1, dt=torch.float32), ro, pool, slot, slot, layout=3, workspace=small)
    assert e.value.status == 5
    assert wpp.wpp_kda_workspace_bytes(1, 1, 4) > 1024
    with pytest.raises(wpp.WppError) as e:                            # periodic snapshots need prefix_lens
        wpp.wpp_kda_chunk(H.ctx(), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128), z(4, 1, 128, dt=torch.float32),
                          z(4, 1, dt=torch.float32), ro, pool, slot, slot, snap_interval=2,
                          snap_slots=torch.zeros(1, 2, dtype=torch.int32, device=dev))
    assert e.value.status == 1


@pytest.mark.parametrize("lanes,chunk", [(8, 2048), (1, 16384)])
def test_full_size_wave_on_sampled_heads(lanes, chunk):
    """The benchmark's waves (8 lanes x 2,048 tokens: one CTA per pair; one lane x 16,384 tokens: the library picks
    four column slices per pair), 32 heads, resumed states: the oracle recomputes sampled (request, head) chains and
    all of their outputs and final states are compared."""
    w = W.kda_wave(lanes, chunk)
    t = w.tensors()
    got_o, got_pool, status = _gpu(w, t)
    assert status == 0
    rows = w.row_offsets
    for req, head in (((0, 0), (3, 17), (7, 31)) if lanes == 8 else ((0, 5),)):
        sl = slice(rows[req], rows[req + 1])
        sub = W.kda_workload("one", 0, [int(w.chunk_lens[req])], 1, [int(w.prefix_lens[req])])
        sub.num_slots, sub.state_in, sub.state_out = w.num_slots, w.state_in[req:req + 1], w.state_out[req:req + 1]
        ts = {k: (v[sl] if k != "state_pool" else v) for k, v in t.items()}
        ref_o, ref_pool = _oracle(sub, ts, heads=slice(head, head + 1))
        _close_out(got_o[sl, head:head + 1], ref_o, f"outputs of request {req} head {head}")
        _close_state(got_pool[w.state_out[req], head], ref_pool[w.state_out[req], 0], "final state")


@pytest.mark.parametrize("seed", range(24))
def test_random_waves_in_the_chunk_parallel_form(seed):
    """Seeded random waves for the chunk-parallel form: chunk lengths around the block size, prefixes at every
    alignment, snapshot intervals from 1 (every token is a sub-block of its own) to beyond a block, some channels with
    zero and tiny decays (extra cuts), odd head counts, resumed and zero states - all against the oracle."""
    rng = np.random.default_rng(4000 + seed)
    R = int(rng.integers(1, 6))
    H_ = int(rng.choice([1, 2, 3]))
    lens = [int(x) for x in rng.choice([0, 1, 2, 31, 63, 64, 65, 100, 127, 128, 129, 200, 333], R)]
    if sum(lens) == 0:
        lens[0] = 70
    prefix = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 100, 128, 1000, 4097], R)]
    interval = int(rng.choice([0, 0, 1, 2, 3, 16, 50, 64, 65, 200]))
    w = W.kda_workload("fuzz", 100 + seed, lens, H_, prefix, resume=rng.random(R) < 0.7, snap_interval=interval)
    t = w.tensors()
    if seed % 3 == 0 and w.total_tokens > 0:
        a = t["alpha"].numpy()
        T = a.shape[0]
        for val, count in ((0.0, 6), (1e-9, 6), (1e-30, 4), (0.2, 200)):
            idx = (rng.integers(0, T, count), rng.integers(0, H_, count), rng.integers(0, 128, count))
            a[idx] = val
    ref_o, ref_pool = _oracle(w, t)
    got_o, got_pool, status = _gpu(w, t, layout=3)
    assert status == 0 and np.isfinite(got_o).all() and np.isfinite(got_pool).all()
    _close_out(got_o, ref_o, "outputs")
    _close_state(got_pool, ref_pool, "state pool")
