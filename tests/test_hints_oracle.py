"""Pins for the oracle of the chained block hash and the hint-index probe (Section 4.3)."""
import numpy as np

from oracle import hints as O


def test_mix64_is_the_published_splitmix64_finaliser():
    # splitmix64 seeded with 0: the state is advanced by the golden-ratio increment and then finalised; its first
    # three outputs are widely published test values
    gamma, state, outs = 0x9E3779B97F4A7C15, 0, []
    for _ in range(3):
        state = (state + gamma) & O.MASK
        outs.append(O.mix64(state))
    assert outs == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_chain_structure_of_eq_design_hash():
    rng = np.random.default_rng(0)
    toks = rng.integers(0, 50000, 5 * 16 + 7).tolist()          # five full blocks and a partial one
    h = O.chained_hashes(toks, 16, salt=3)
    assert len(h) == 5 and len(set(h)) == 5                      # only full blocks; all distinct
    # a key depends on its own block and, through the parent hash, on every block before it - and on nothing after
    other = list(toks)
    other[2 * 16 + 5] += 1
    g = O.chained_hashes(other, 16, salt=3)
    assert g[:2] == h[:2] and all(a != b for a, b in zip(g[2:], h[2:]))
    # order inside a block matters, and so do salt and extra keys
    swapped = list(toks)
    swapped[0], swapped[1] = swapped[1], swapped[0]
    assert O.chained_hashes(swapped, 16, salt=3)[0] != h[0]
    assert O.chained_hashes(toks, 16, salt=4)[0] != h[0]
    assert O.chained_hashes(toks, 16, salt=3, extra_keys=[0, 0, 9, 0, 0])[:2] == h[:2]
    assert O.chained_hashes(toks, 16, salt=3, extra_keys=[0, 0, 9, 0, 0])[2] != h[2]
    # H_{-1} = 0: the first key is the hash of the first block with parent 0 (recomputed here by hand)
    s = (3 * 0x9E3779B97F4A7C15) & O.MASK
    assert h[0] == O.mix64(0 ^ O.mix64(O.block_digest(toks[:16])) ^ s)
    # two requests with a common prefix share exactly the keys of the common full blocks
    fork = toks[:3 * 16] + rng.integers(0, 50000, 40).tolist()
    f = O.chained_hashes(fork, 16, salt=3)
    assert f[:3] == h[:3] and f[3] != h[3]
    assert O.chained_hashes([], 16) == [] and O.chained_hashes(toks[:15], 16) == []


def test_counted_index_follows_blocks_joining_and_leaving_the_tree():
    idx = O.HintIndex()
    idx.add(0, [11, 12, 13])
    idx.add(0, [11, 12])                   # a second sequence shares the first two blocks
    idx.add(1, [11])                       # another cache window is another key
    assert len(idx) == 4 and idx.has(0, 13) and idx.has(1, 11) and not idx.has(1, 12)
    idx.remove(0, [11, 12, 13])
    assert idx.has(0, 11) and idx.has(0, 12) and not idx.has(0, 13)        # counters 1, 1, gone
    idx.remove(0, [11, 12])
    assert len(idx) == 1
    idx.remove(0, [11])                    # removing what is not there changes nothing
    assert len(idx) == 1


def test_figure_example_gallop_and_bisect_to_seven_blocks():
    # Figure "sharded hint index": the attention probe gallops and bisects to seven blocks
    toks = list(range(12 * 16))
    h = O.chained_hashes(toks, 16)
    idx = O.HintIndex()
    idx.add(0, h[:7])
    depth, probed = O.probe_gallop_bisect(idx, 0, h)
    assert depth == 7 and probed == [1, 2, 4, 8, 6, 7]          # 1 2 4 hit, 8 misses, then 6 and 7


def test_probe_equals_the_linear_definition_with_logarithmically_many_probes():
    rng = np.random.default_rng(1)
    for _ in range(400):
        N = int(rng.integers(0, 200))
        hashes = [int(x) for x in rng.integers(1, 1 << 62, N)]
        m = int(rng.integers(0, N + 1))
        idx = O.HintIndex()
        idx.add(7, hashes[:m])
        idx.add(8, hashes)                                      # another window must not matter
        depth, probed = O.probe_gallop_bisect(idx, 7, hashes)
        assert depth == m == O.longest_prefix_linear(idx, 7, hashes)
        assert len(probed) <= 2 * max(1, N).bit_length() + 1 and len(set(probed)) == len(probed)
    # edge cases: nothing eligible, nothing cached, everything cached (no miss is ever seen)
    idx = O.HintIndex()
    assert O.probe_gallop_bisect(idx, 0, []) == (0, [])
    assert O.probe_gallop_bisect(idx, 0, [5, 6, 7]) == (0, [1])
    idx.add(0, [5, 6, 7, 8, 9])
    assert O.probe_gallop_bisect(idx, 0, [5, 6, 7, 8, 9]) == (5, [1, 2, 4, 5])


def test_reverse_scan_finds_the_deepest_snapshot_at_or_below_the_attention_endpoint():
    # the definition: max depth d <= limit with the key present (brute force over all depths), 0 if none
    rng = np.random.default_rng(2)
    for _ in range(300):
        N = int(rng.integers(0, 120))
        hashes = [int(x) for x in rng.integers(1, 1 << 62, N)]
        snaps = sorted(set(int(d) for d in rng.integers(1, N + 1, rng.integers(0, 6)))) if N else []
        idx = O.HintIndex()
        idx.add(3, [hashes[d - 1] for d in snaps])
        idx.add(0, hashes)                                      # the attention window holds every block; must not matter
        limit = int(rng.integers(0, N + 1))
        want = max([d for d in snaps if d <= limit], default=0)
        depth, probed = O.probe_reverse_scan(idx, 3, hashes, limit)
        assert depth == want
        assert probed == list(range(limit, max(want, 1) - 1, -1))          # limit, limit-1, ..., down to the hit (or 1)
    # Section 4.4's example in blocks: snapshots at 64K, 72K, 90K tokens; an attention endpoint of 80K falls back to 72K
    B, toks = 1024, list(range(96 * 1024))
    h = O.chained_hashes(toks, B)
    idx = O.HintIndex()
    idx.add(1, [h[64 - 1], h[72 - 1], h[90 - 1]])
    assert O.probe_reverse_scan(idx, 1, h, 80)[0] == 72 and O.probe_reverse_scan(idx, 1, h, 71)[0] == 64
    assert O.probe_reverse_scan(idx, 1, h, 63)[0] == 0 and O.reuse_candidate([80, 72]) == 72
