"""Oracle for the wave-budget planner and FCFS packing of Section 4.5 ("Pipeline Scheduling", MPU).

TEST INFRASTRUCTURE ONLY: plain Python integers and fractions, written from the paper's formulas in the paper's
notation; it shares no code with the C implementation (`wpp_plan_waves`) and only tests and bench.py's CPU legs
import it.

Notation (Section 4.5): P pipeline stages; execution ring of R = 2P waves; fill factor F; target S = R + (F-1)P
waves; block size B; maximum wave budget M and floor b_min (both multiples of B, B <= b_min <= M).  `pieces` are
the not-yet-scheduled suffixes of admitted requests together with their most recently committed chunks that are
still in the ring; W is their token sum.

Where the paper leaves a rule open, the reading taken here is marked "READING";
those parts are pinned only by examples constructed from the reading: parity unpinned for them.
"""
from fractions import Fraction


def budget_ladder(M, b_min, B):
    """Eq. (design-budget): b_0 = M, b_{j+1} = max(b_min, alignDown_B(b_j / 2)); halving stops at b_min."""
    assert B > 0 and M % B == 0 and b_min % B == 0 and B <= b_min <= M
    ladder = [M]
    while ladder[-1] > b_min:
        half = ladder[-1] // 2
        ladder.append(max(b_min, (half // B) * B))
    return ladder


def ring_and_target(P, F):
    """R = 2P waves in the execution ring; the planner aims at S = R + (F - 1) P waves."""
    R = 2 * P
    return R, R + (F - 1) * P


def available_waves(b, pieces):
    """n(b) = max(W / b, N_{>b/2}): token count alone underestimates the waves when pieces larger than half a
    wave cannot share one.  Returned as an exact fraction."""
    W = sum(pieces)
    n_big = sum(1 for p in pieces if 2 * p > b)
    return max(Fraction(W, b), Fraction(n_big))


def newly_split_tokens(b_large, b_small, pieces):
    """Tokens in pieces that fit the larger budget whole but would have to be split under the smaller one."""
    return sum(p for p in pieces if b_small < p <= b_large)


def select_budget(ladder, R, S, pieces):
    """Index of the budget the paper's rule selects, before hysteresis.

    Walk down the ladder from M: the first (largest) budget with n(b) >= S wins; b_min if none does.  Thinning
    limit: once a budget already supplies R waves, the next smaller one is taken only if the pieces it would
    newly split make up at most 12.5 % of W.
    READING: "newly split" = pieces of size in (b_{j+1}, b_j]; the limit is tested at every step down whose upper
    budget has n(b_j) >= R."""
    W = sum(pieces)
    j = 0
    while j + 1 < len(ladder) and available_waves(ladder[j], pieces) < S:
        if available_waves(ladder[j], pieces) >= R and 8 * newly_split_tokens(ladder[j], ladder[j + 1], pieces) > W:
            break
        j += 1
    return j


class BudgetState:
    """Budget in force (index into the ladder) and the pending change: direction (-1 towards larger budgets,
    +1 towards smaller, 0 none) and for how many consecutive decisions it has been asked for."""

    def __init__(self, cur=0, direction=0, count=0):
        self.cur, self.direction, self.count = cur, direction, count

    def as_tuple(self):
        return (self.cur, self.direction, self.count)


def apply_hysteresis(state, target, ladder, R, S, pieces):
    """One planning decision: move `state.cur` towards `target` under the paper's persistence rules.

    - A burst that asks for a budget two or more ladder steps larger takes effect at once.
    - A one-step increase must have been asked for by R/2 consecutive decisions.
    - A decrease must have been asked for by R consecutive decisions and pass a hysteresis check.
    READING: a change moves one ladder step at a time (except the burst); "consecutive" is reset by any decision
    that asks for no change or for the other direction; the hysteresis check (not specified in the paper) is that
    the budget in force misses the target by at least one whole wave, n(b_cur) <= S - 1."""
    cur = state.cur
    if target == cur:
        return BudgetState(cur, 0, 0)
    if target < cur:                                   # larger budget wanted
        if cur - target >= 2:
            return BudgetState(target, 0, 0)
        count = state.count + 1 if state.direction == -1 else 1
        if count >= R // 2:
            return BudgetState(cur - 1, 0, 0)
        return BudgetState(cur, -1, count)
    count = state.count + 1 if state.direction == +1 else 1      # smaller budget wanted
    if count >= R and available_waves(ladder[cur], pieces) <= S - 1:
        return BudgetState(cur + 1, 0, 0)
    return BudgetState(cur, +1, count)


def pack_wave(b, b_min, remaining, max_lanes):
    """Rank 0 packs requests in FCFS order into one wave of at most b tokens and max_lanes requests.

    A request that fits takes all its remaining tokens.  One that does not fit gets the leftover space as a
    fragment, unless that fragment is smaller than max(b_min, b/2): small leftovers are not filled with a piece of
    a larger request.
    READING: packing stops at the first request that cannot be placed (FCFS order is not overtaken)."""
    chunks = [0] * len(remaining)
    space, lanes = b, 0
    for i, r in enumerate(remaining):
        if r == 0:
            continue
        if lanes == max_lanes or space == 0:
            break
        if r <= space:
            take = r
        else:
            if 2 * space < max(2 * b_min, b):
                break
            take = space
        chunks[i] = take
        space -= take
        lanes += 1
    return chunks


def plan_wave(P, F, M, b_min, B, max_lanes, remaining, inflight, state, ring_busy=False, admission_pending=False,
              already_deferred=False):
    """One planning decision of rank 0: budget (with hysteresis), then the wave's chunks.

    remaining: not-yet-scheduled suffix tokens per admitted request, FCFS order.  inflight: most recently committed
    chunks still in the ring.  Returns (new_state, budget, chunk_lens, defer) where `defer` says the wave is a lone
    request below half capacity that may wait one iteration for company while the ring is busy."""
    ladder = budget_ladder(M, b_min, B)
    R, S = ring_and_target(P, F)
    pieces = [r for r in remaining if r > 0] + [c for c in inflight if c > 0]
    target = select_budget(ladder, R, S, pieces)
    new_state = apply_hysteresis(state, target, ladder, R, S, pieces)
    b = ladder[new_state.cur]
    chunks = pack_wave(b, b_min, remaining, max_lanes)
    lanes = sum(1 for c in chunks if c > 0)
    defer = bool(ring_busy and admission_pending and not already_deferred and lanes == 1 and 2 * sum(chunks) < b)
    return new_state, b, chunks, defer
