"""wpp_plan_waves (C, through the C ABI) against the oracle of Section 4.5: bit-exact on every output, over seeded
random queues, long decision sequences with carried state, and the edge cases.  No GPU involved: the planner is
host code."""
import numpy as np
import pytest

import paper_2609_35263_b200 as wpp
from oracle import waves as O


def _cfg(P, F, B, lanes, M, b_min):
    return wpp.WaveConfig(P, F, B, lanes, M, b_min)


def _decide(cfg, state, ostate, remaining, inflight, flags=0):
    chunks, info = wpp.wpp_plan_waves(cfg, state, remaining, inflight, flags)
    o_state, o_b, o_chunks, o_defer = O.plan_wave(
        cfg.num_stages, cfg.fill_factor, cfg.max_budget, cfg.min_budget, cfg.block_size, cfg.max_lanes,
        list(remaining), list(inflight), ostate, ring_busy=bool(flags & 1), admission_pending=bool(flags & 2),
        already_deferred=bool(flags & 4))
    ladder = O.budget_ladder(cfg.max_budget, cfg.min_budget, cfg.block_size)
    R, S = O.ring_and_target(cfg.num_stages, cfg.fill_factor)
    pieces = [r for r in remaining if r > 0] + [c for c in inflight if c > 0]
    assert chunks.tolist() == o_chunks
    assert state.as_tuple() == o_state.as_tuple()
    assert int(info.budget) == o_b == ladder[o_state.cur] and int(info.budget_index) == o_state.cur
    assert int(info.target_index) == O.select_budget(ladder, R, S, pieces)
    assert int(info.work) == sum(pieces) and int(info.wave_tokens) == sum(o_chunks)
    assert int(info.lanes) == sum(1 for c in o_chunks if c) and bool(info.defer) == o_defer
    return chunks, o_state


@pytest.mark.parametrize("P,F,B,lanes,M,b_min", [
    (4, 2, 64, 8, 16384, 8192),          # the paper's matched PP4 settings
    (4, 2, 64, 64, 16384, 1024),
    (1, 1, 16, 2, 1024, 16),
    (8, 3, 128, 16, 32768, 2048),
    (2, 2, 64, 4, 10048, 64),            # budgets that are not powers of two
])
def test_ladder_matches(P, F, B, lanes, M, b_min):
    assert wpp.wpp_wave_ladder(_cfg(P, F, B, lanes, M, b_min)) == O.budget_ladder(M, b_min, B)


@pytest.mark.parametrize("seed", range(6))
def test_single_decisions_on_random_queues(seed):
    rng = np.random.default_rng(seed)
    for _ in range(300):
        B = int(rng.choice([16, 64, 128]))
        b_min = B * int(rng.integers(1, 33))
        M = b_min * int(rng.integers(1, 17))
        M -= M % B
        cfg = _cfg(int(rng.integers(1, 9)), int(rng.integers(1, 4)), B, int(rng.integers(1, 10)), M, b_min)
        L = len(O.budget_ladder(M, b_min, B))
        cur = int(rng.integers(0, L))
        direction = int(rng.integers(-1, 2))
        count = int(rng.integers(0, 20)) if direction else 0
        n = int(rng.integers(0, 30))
        scale = int(rng.choice([B, M // 4 + 1, 3 * M]))
        remaining = [int(x) if rng.random() > 0.15 else 0 for x in rng.integers(0, scale + 1, n)]
        inflight = [int(x) for x in rng.integers(0, M + 1, rng.integers(0, 6))]
        st = wpp.WaveState(cur, direction, count, 0)
        _decide(cfg, st, O.BudgetState(cur, direction, count), remaining, inflight, int(rng.integers(0, 8)))


def test_a_long_run_with_carried_state_drains_the_queue_identically():
    """A serving-like loop: requests arrive in bursts, every decision schedules one wave, accepted spans leave the
    queue, the chunks scheduled last stay in flight for R decisions.  Both planners must walk the same path."""
    rng = np.random.default_rng(42)
    cfg = _cfg(4, 2, 64, 8, 16384, 1024)
    R, _ = O.ring_and_target(4, 2)
    st, ost = wpp.WaveState(), O.BudgetState()
    queue, ring, seen_budgets, scheduled = [], [], set(), 0
    for it in range(900):
        if it < 450 and rng.random() < 0.15:
            queue += [int(x) for x in rng.integers(1, 30000, rng.integers(1, 6))]
        inflight = [c for wave in ring for c in wave]
        chunks, ost = _decide(cfg, st, ost, queue, inflight, flags=int(rng.integers(0, 8)))
        seen_budgets.add(st.cur)
        wave = [int(c) for c in chunks if c]
        scheduled += sum(wave)
        queue = [r - int(c) for r, c in zip(queue, chunks)]
        queue = [r for r in queue if r > 0] if rng.random() < 0.5 else queue      # finished requests may linger as zeros
        ring = (ring + [wave])[-R:]
    assert not [r for r in queue if r > 0] and scheduled > 0                      # everything was scheduled
    assert len(seen_budgets) >= 3                                                 # the budget really moved


def test_edge_cases_and_errors():
    cfg = _cfg(2, 2, 64, 4, 4096, 1024)
    st = wpp.WaveState()
    chunks, info = wpp.wpp_plan_waves(cfg, st, [], [])                            # nothing admitted
    assert chunks.size == 0 and info.lanes == 0 and info.work == 0 and info.wave_tokens == 0
    _decide(cfg, wpp.WaveState(), O.BudgetState(), [0, 0, 0], [])                 # only finished requests
    _decide(cfg, wpp.WaveState(), O.BudgetState(), [10 ** 9], [])                 # one huge request: a full wave
    _decide(cfg, wpp.WaveState(), O.BudgetState(), [700], [], flags=3)            # lone small wave: defer
    _decide(cfg, wpp.WaveState(), O.BudgetState(), [700], [], flags=7)            # ... once only
    for bad in (_cfg(0, 2, 64, 4, 4096, 1024), _cfg(2, 0, 64, 4, 4096, 1024), _cfg(2, 2, 0, 4, 4096, 1024),
                _cfg(2, 2, 64, 0, 4096, 1024), _cfg(2, 2, 64, 4, 4100, 1024), _cfg(2, 2, 64, 4, 4096, 1000),
                _cfg(2, 2, 64, 4, 1024, 4096), _cfg(2, 2, 64, 4, 4096, 0)):
        with pytest.raises(wpp.WppError) as e:
            wpp.wpp_plan_waves(bad, wpp.WaveState(), [100], [])
        assert e.value.status == 1
    with pytest.raises(wpp.WppError):
        wpp.wpp_plan_waves(cfg, wpp.WaveState(9, 0, 0, 0), [100], [])             # state outside the ladder
    with pytest.raises(wpp.WppError):
        wpp.wpp_plan_waves(cfg, wpp.WaveState(), [-5], [])                        # negative length


def test_chunk_lens_feed_the_tile_planner():
    """The planner's output is the chunk_lens argument of the attention path: plan tiles for the wave it made."""
    cfg = _cfg(4, 2, 64, 8, 16384, 8192)
    remaining = [20000, 3000, 500, 9000]
    prefix = [16384, 0, 128, 4096]                                                # tokens already cached per request
    chunks, info = wpp.wpp_plan_waves(cfg, wpp.WaveState(), remaining, [])
    assert chunks.tolist() == [16384, 0, 0, 0] and info.budget == 16384          # FCFS: the first request fills the wave
    mb = max((p + int(c) + 63) // 64 for p, c in zip(prefix, chunks))
    desc = wpp.make_desc(len(remaining), 16, 4, 128, 64, mb, 4096)
    plan = wpp.wpp_plan_tiles(None, desc, prefix, chunks.tolist(), pin=False)
    assert plan.info.total_new_tokens == int(chunks.sum()) and plan.info.num_tiles > 0
