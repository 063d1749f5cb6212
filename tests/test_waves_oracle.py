"""Pins for the wave-budget oracle (Section 4.5): the paper's own numbers and examples, closed forms and
hand-worked cases, chosen so that a dropped term or an off-by-one in any rule fails one of them."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import waves as O


def test_ladder_of_the_matched_pp4_settings_has_two_budgets():
    # Section 4.5: "The matched PP4 comparison uses M = 16,384 and b_min = 8,192"
    assert O.budget_ladder(16384, 8192, 64) == [16384, 8192]


def test_ladder_halves_aligns_down_and_stops_at_the_floor():
    assert O.budget_ladder(16384, 1024, 64) == [16384, 8192, 4096, 2048, 1024]
    # 157 blocks of 64: every halving is rounded down to whole blocks, the floor is reached exactly once
    # 5024 -> 78 blocks, 2496 = 39 blocks, 1248 -> 19 blocks, 608 -> 9 blocks, 288 -> 4 blocks
    assert O.budget_ladder(10048, 64, 64) == [10048, 4992, 2496, 1216, 576, 256, 128, 64]
    assert O.budget_ladder(4096, 4096, 64) == [4096]
    # a floor that is not on the halving path still ends the ladder
    assert O.budget_ladder(4096, 1536, 512) == [4096, 2048, 1536]


def test_ring_and_target_of_the_matched_experiments():
    # R = 2P, S = R + (F - 1) P; "The matched PP4 experiments use F = 2"
    assert O.ring_and_target(4, 2) == (8, 12)
    assert O.ring_and_target(1, 1) == (2, 2)
    assert O.ring_and_target(8, 3) == (16, 32)


def test_figure_example_two_budgets_of_tokens_give_two_waves_or_four():
    # Figure "Wave sizing with the same 2M tokens on four stages": budget M -> two waves, M/2 -> four
    M = 16384
    pieces = [2048] * 16                       # 2M tokens in pieces that share waves freely
    assert O.available_waves(M, pieces) == 2
    assert O.available_waves(M // 2, pieces) == 4


def test_pieces_larger_than_half_a_wave_cannot_share_one():
    b = 1000
    pieces = [600] * 5                         # W / b = 3, but no two of them fit one wave
    assert O.available_waves(b, pieces) == 5
    assert O.available_waves(b, [500] * 6) == 3            # exactly half does share
    assert O.available_waves(b, [501] + [1] * 10) == 1                  # W / b = 0.511, one piece above half
    assert O.available_waves(b, [499] + [1] * 10) == Fraction(509, 1000)
    assert O.available_waves(b, []) == 0


def test_selection_takes_the_largest_budget_that_supplies_s_waves():
    ladder = O.budget_ladder(1024, 128, 64)                # 1024 512 256 128
    R, S = O.ring_and_target(1, 1)                         # 2, 2
    assert O.select_budget(ladder, R, S, [64] * 32) == 0   # W = 2048 = 2 M
    assert O.select_budget(ladder, R, S, [64] * 24) == 1   # 1.5 M: n(M) = 1.5, n(M/2) = 3
    assert O.select_budget(ladder, R, S, [64] * 9) == 2    # 576: n(512) = 1.125, n(256) = 2.25
    assert O.select_budget(ladder, R, S, [64] * 3) == 3    # nothing qualifies: the floor
    assert O.select_budget(ladder, R, S, []) == 3
    # boundary: n(b) >= S is inclusive
    assert O.select_budget(ladder, R, S, [64] * 16) == 1   # W = 1024: n(1024) = 1 < 2, n(512) = 2


def test_thinning_limit_of_one_eighth():
    ladder = O.budget_ladder(1024, 256, 64)                # 1024 512 256
    R, S = O.ring_and_target(1, 3)                         # 2, 4
    # M already supplies R = 2 waves; going to 512 would split the two pieces of 1000 = 95 % of W: stay at M
    assert O.select_budget(ladder, R, S, [1000, 1000, 100]) == 0
    # same amount of work in small pieces: nothing is newly split, 512 supplies 4.1 waves
    assert O.select_budget(ladder, R, S, [100] * 21) == 1
    # newly split pieces exactly one eighth of W are still allowed ("at most 12.5 %")
    pieces = [600] + [100] * 42                            # W = 4800, 600 = W / 8; n(1024) = 4.69 >= S anyway
    assert O.select_budget(ladder, R, S, pieces) == 0
    pieces = [600] + [75] * 28                             # W = 2700: n(1024) = 2.64 in [R, S); 600 > 2700 / 8
    assert O.select_budget(ladder, R, S, pieces) == 0
    pieces = [300] + [75] * 28                             # W = 2400: 300 = W / 8 is allowed, but it is not newly
    assert O.select_budget(ladder, R, S, pieces) == 1      # split at 512 anyway; n(512) = 4.69
    # the limit only applies once the larger budget supplies R waves
    assert O.select_budget(ladder, R, S, [100] * 5) == 2   # n(1024) = 0.49, n(512) = 0.98: both below R, on to the floor
    # two pieces above half of M already make R = 2 waves of it (N counts, not W / b = 1.86): both would be split
    assert O.select_budget(ladder, R, S, [1000, 900]) == 0
    # n(1024) = 1.37 < R: one step down is free; 512 supplies 2.73 >= R and the 400 would be newly split at 256
    assert O.select_budget(ladder, R, S, [1000, 400]) == 1


def test_newly_split_counts_pieces_between_the_two_budgets():
    assert O.newly_split_tokens(1024, 512, [512, 513, 1024, 1025, 10]) == 513 + 1024


def test_hysteresis_increase_needs_half_a_ring_of_decisions_unless_it_is_a_burst():
    ladder = O.budget_ladder(4096, 512, 64)                # 4096 2048 1024 512
    R, S = O.ring_and_target(2, 2)                         # 4, 6
    st = O.BudgetState(cur=2)
    # one step up must be asked for by R/2 = 2 consecutive decisions
    st = O.apply_hysteresis(st, 1, ladder, R, S, [])
    assert st.as_tuple() == (2, -1, 1)
    st = O.apply_hysteresis(st, 1, ladder, R, S, [])
    assert st.as_tuple() == (1, 0, 0)
    # an interruption resets the count
    st = O.BudgetState(cur=2)
    st = O.apply_hysteresis(st, 1, ladder, R, S, [])
    st = O.apply_hysteresis(st, 2, ladder, R, S, [])
    st = O.apply_hysteresis(st, 1, ladder, R, S, [])
    assert st.as_tuple() == (2, -1, 1)
    # a burst (two or more steps) takes effect at once
    assert O.apply_hysteresis(O.BudgetState(cur=3), 0, ladder, R, S, []).as_tuple() == (0, 0, 0)
    assert O.apply_hysteresis(O.BudgetState(cur=2), 0, ladder, R, S, []).as_tuple() == (0, 0, 0)


def test_hysteresis_decrease_needs_a_full_ring_of_decisions_and_a_margin():
    ladder = O.budget_ladder(4096, 512, 64)
    R, S = O.ring_and_target(2, 2)                         # 4, 6
    few = [64] * 8                                         # W = 512: n(4096) = 0.125 <= S - 1
    st = O.BudgetState(cur=0)
    for i in range(3):
        st = O.apply_hysteresis(st, 3, ladder, R, S, few)
        assert st.as_tuple() == (0, +1, i + 1)
    st = O.apply_hysteresis(st, 3, ladder, R, S, few)      # fourth consecutive decision: one step down
    assert st.as_tuple() == (1, 0, 0)
    # without the margin (n(b_cur) > S - 1) the decrease keeps waiting
    near = [64] * 336                                      # W = 21504: n(4096) = 5.25 > 5
    st = O.BudgetState(cur=0, direction=+1, count=10)
    st = O.apply_hysteresis(st, 1, ladder, R, S, near)
    assert st.as_tuple() == (0, +1, 11)
    # a change of direction restarts the count
    st = O.apply_hysteresis(O.BudgetState(cur=1, direction=+1, count=3), 0, ladder, R, S, few)
    assert st.as_tuple() == (1, -1, 1)


def test_packing_is_fcfs_with_the_fragment_rule():
    # everything fits
    assert O.pack_wave(1024, 256, [300, 200, 100], 8) == [300, 200, 100]
    # leftover 524 >= max(b_min, b/2) = 512: the next request is split
    assert O.pack_wave(1024, 256, [500, 900], 8) == [500, 524]
    # leftover 424 < 512: not filled with a fragment of the larger request, and nobody overtakes it
    assert O.pack_wave(1024, 256, [600, 900, 50], 8) == [600, 0, 0]
    # the fragment threshold is max(b_min, b/2): with a high floor even 700 left is not enough
    assert O.pack_wave(1024, 768, [324, 900], 8) == [324, 0]
    assert O.pack_wave(1024, 768, [256, 900], 8) == [256, 768]
    # an oversized first request takes the whole wave
    assert O.pack_wave(1024, 256, [5000, 10], 8) == [1024, 0]
    # lanes limit and finished requests
    assert O.pack_wave(1024, 256, [10, 0, 10, 10, 10], 3) == [10, 0, 10, 10, 0]
    assert O.pack_wave(1024, 256, [], 4) == []


def test_packing_invariants_on_random_queues():
    rng = np.random.default_rng(0)
    for _ in range(300):
        b_min = int(rng.integers(1, 9)) * 64
        b = b_min * int(rng.integers(1, 9))
        remaining = [int(x) for x in rng.integers(0, 3 * b, rng.integers(0, 12))]
        lanes = int(rng.integers(1, 6))
        chunks = O.pack_wave(b, b_min, remaining, lanes)
        assert len(chunks) == len(remaining) and sum(chunks) <= b
        assert sum(1 for c in chunks if c) <= lanes
        assert all(0 <= c <= r for c, r in zip(chunks, remaining))
        live = [i for i, r in enumerate(remaining) if r]
        taken = [i for i, c in enumerate(chunks) if c]
        assert taken == live[:len(taken)]                              # FCFS: a prefix of the waiting requests
        for k, i in enumerate(taken):
            if chunks[i] < remaining[i]:                               # a fragment: last in the wave and not small
                assert k == len(taken) - 1 and 2 * chunks[i] >= max(2 * b_min, b)


def test_plan_wave_worked_example():
    # P = 2 stages, F = 2: R = 4, S = 6.  M = 4096, floor 1024, blocks of 64.
    st = O.BudgetState(cur=0)
    remaining = [3000, 500, 2000]                                      # W = 5500 + 1000 in flight
    st2, b, chunks, defer = O.plan_wave(2, 2, 4096, 1024, 64, 4, remaining, [1000], st)
    # n(4096) = 1.59 < S; 4096 does not supply R either, so thinning goes on: n(2048) = 3.17, n(1024) = 6.35 -> floor
    # wanted, but a decrease needs R = 4 consecutive decisions: the budget in force stays M for now
    assert st2.as_tuple() == (0, +1, 1) and b == 4096
    assert chunks == [3000, 500, 0] and defer is False                 # 596 left < 2048: no fragment of the third
    lone = O.plan_wave(2, 2, 4096, 1024, 64, 4, [700], [], O.BudgetState(cur=0), ring_busy=True,
                       admission_pending=True)
    assert lone[2] == [700] and lone[3] is True                        # a lone wave below half capacity may wait
    again = O.plan_wave(2, 2, 4096, 1024, 64, 4, [700], [], O.BudgetState(cur=0), ring_busy=True,
                        admission_pending=True, already_deferred=True)
    assert again[3] is False                                           # ... one iteration only


@pytest.mark.parametrize("P,F", [(1, 1), (2, 2), (4, 2), (8, 3)])
def test_selected_budget_supplies_s_waves_or_is_pinned_by_a_rule(P, F):
    """Whatever the rules decide, the result is explainable: either the budget supplies S waves and the next larger
    one does not, or it is the floor, or the thinning limit stopped the walk."""
    rng = np.random.default_rng(P * 10 + F)
    ladder = O.budget_ladder(16384, 1024, 64)
    R, S = O.ring_and_target(P, F)
    for _ in range(400):
        pieces = [int(x) for x in rng.integers(1, 20000, rng.integers(0, 40))]
        j = O.select_budget(ladder, R, S, pieces)
        W = sum(pieces)
        for i in range(j):                                             # every larger budget was passed over legally
            assert O.available_waves(ladder[i], pieces) < S
            if O.available_waves(ladder[i], pieces) >= R:
                assert 8 * O.newly_split_tokens(ladder[i], ladder[i + 1], pieces) <= W
        if O.available_waves(ladder[j], pieces) < S and j + 1 < len(ladder):
            assert O.available_waves(ladder[j], pieces) >= R
            assert 8 * O.newly_split_tokens(ladder[j], ladder[j + 1], pieces) > W
