"""Chained block hashes and the hint index of the library against the oracle of Section 4.3: bit-exact hashes (host
entry point here, GPU kernels in the gpu-marked test), identical index contents, identical probe results and probe
counts."""
import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
from oracle import hints as O


def _requests(rng, n, B, vocab=150000, max_blocks=40):
    lens = [int(rng.integers(0, max_blocks * B)) for _ in range(n)]
    return [rng.integers(0, vocab, L).astype(np.int32) for L in lens]


@pytest.mark.parametrize("B", [16, 64, 33])
def test_host_hashes_match_the_oracle(B):
    rng = np.random.default_rng(B)
    for toks in _requests(rng, 20, B):
        n = len(toks) // B
        extra = rng.integers(0, 1 << 62, n).astype(np.uint64) if rng.random() < 0.5 else None
        salt = int(rng.integers(0, 1 << 62))
        got = wpp.wpp_hash_blocks_host(toks, B, salt, extra)
        want = O.chained_hashes(toks.tolist(), B, salt, None if extra is None else extra.tolist())
        assert got.tolist() == want
    assert wpp.wpp_hash_blocks_host(np.array([-1, 2 ** 31 - 1] * 8, dtype=np.int32), 16).tolist() == \
        O.chained_hashes([-1, 2 ** 31 - 1] * 8, 16)                                    # negative ids wrap mod 2^32
    assert wpp.wpp_hash_blocks_host([], 16).size == 0


def test_index_and_probe_match_the_oracle_on_a_churning_cache():
    rng = np.random.default_rng(3)
    B = 16
    idx, oidx = wpp.HintIndex(), O.HintIndex()
    base = rng.integers(0, 1000, 30 * B).astype(np.int32)                              # a popular prefix
    live = []
    for it in range(300):
        # a request: some prefix of the popular one, then its own tokens
        keep = int(rng.integers(0, 31)) * B
        toks = np.concatenate([base[:keep], rng.integers(0, 1000, int(rng.integers(0, 20 * B))).astype(np.int32)])
        window = int(rng.integers(0, 2))
        h = wpp.wpp_hash_blocks_host(toks, B, salt=9)
        assert h.tolist() == O.chained_hashes(toks.tolist(), B, 9)
        got = idx.probe(window, h)
        want_depth, want_probed = O.probe_gallop_bisect(oidx, window, h.tolist())
        assert got == (want_depth, len(want_probed))
        assert want_depth == O.longest_prefix_linear(oidx, window, h.tolist())
        # the request is admitted: a prefix of its blocks joins the tree; sometimes an older one leaves
        cached = h[:int(rng.integers(0, len(h) + 1))]
        idx.add(window, cached)
        oidx.add(window, cached.tolist())
        live.append((window, cached))
        if len(live) > 12:
            w0, old = live.pop(int(rng.integers(0, len(live))))
            idx.remove(w0, old)
            oidx.remove(w0, old.tolist())
        assert len(idx) == len(oidx)
    for w0, old in live:
        idx.remove(w0, old)
    assert len(idx) == 0
    idx.close()


def test_reverse_scan_matches_the_oracle_and_gives_the_joint_candidate():
    """Attention blocks are dense, recurrent snapshots sparse: the candidate is the minimum of the two endpoints, the
    recurrent one found by scanning backward from the attention one (Section 4.3)."""
    rng = np.random.default_rng(8)
    ATT, REC = 0, 1
    for _ in range(200):
        N = int(rng.integers(0, 150))
        hashes = np.array([int(x) for x in rng.integers(1, 1 << 62, N)], dtype=np.uint64)
        cached = int(rng.integers(0, N + 1))
        snaps = sorted(set(int(d) for d in rng.integers(1, N + 1, rng.integers(0, 5)))) if N else []
        idx, oidx = wpp.HintIndex(), O.HintIndex()
        for i in (idx, oidx):
            i.add(ATT, hashes[:cached].tolist())
            i.add(REC, [int(hashes[d - 1]) for d in snaps])
        att, _ = idx.probe(ATT, hashes)
        assert att == O.probe_gallop_bisect(oidx, ATT, hashes.tolist())[0] == cached
        rec, probes = idx.probe_recurrent(REC, hashes, att)
        want, probed = O.probe_reverse_scan(oidx, REC, hashes.tolist(), att)
        assert (rec, probes) == (want, len(probed))
        assert O.reuse_candidate([att, rec]) == max([d for d in snaps if d <= cached], default=0)
    idx = wpp.HintIndex()
    assert idx.probe_recurrent(REC, [], 0) == (0, 0) and idx.probe_recurrent(REC, [5, 6], 9) == (0, 2)


def test_figure_example_through_the_library():
    h = wpp.wpp_hash_blocks_host(np.arange(12 * 16, dtype=np.int32), 16)
    idx = wpp.HintIndex()
    idx.add(0, h[:7])
    assert idx.probe(0, h) == (7, 6)           # probes 1 2 4 8 6 7
    assert idx.probe(1, h) == (0, 1)           # another cache window knows nothing
    assert idx.probe(0, h[:0]) == (0, 0)
    assert idx.probe(0, h[:7]) == (7, 5)       # 1 2 4 hit, no miss to see, then 6 and 7


def test_matched_blocks_become_prefix_lens_of_the_attention_path():
    """hash -> probe -> prefix_lens -> wave planner -> tile planner: the steps upstream of the kernels in a row."""
    B = 64
    rng = np.random.default_rng(5)
    shared = rng.integers(0, 50000, 16 * B).astype(np.int32)
    idx = wpp.HintIndex()
    idx.add(0, wpp.wpp_hash_blocks_host(shared, B))
    reqs = [np.concatenate([shared, rng.integers(0, 50000, n).astype(np.int32)]) for n in (700, 5000)]
    reqs.append(rng.integers(0, 50000, 3000).astype(np.int32))                         # no reuse
    prefix = [idx.probe(0, wpp.wpp_hash_blocks_host(t, B))[0] * B for t in reqs]
    assert prefix == [16 * B, 16 * B, 0]
    remaining = [len(t) - p for t, p in zip(reqs, prefix)]
    chunks, info = wpp.wpp_plan_waves(wpp.WaveConfig(4, 2, B, 8, 16384, 8192), wpp.WaveState(), remaining, [])
    assert chunks.tolist() == remaining and info.wave_tokens == sum(remaining)
    mb = max((p + c + B - 1) // B for p, c in zip(prefix, chunks.tolist()))
    plan = wpp.wpp_plan_tiles(None, wpp.make_desc(3, 16, 4, 128, B, mb, 1024), prefix, chunks.tolist(), pin=False)
    assert plan.info.total_new_tokens == sum(remaining)


@pytest.mark.gpu
@pytest.mark.parametrize("B", [16, 64, 48])
def test_gpu_hashes_match_the_oracle(B):
    rng = np.random.default_rng(100 + B)
    reqs = _requests(rng, 37, B, max_blocks=70) + [np.zeros(0, dtype=np.int32), np.arange(B - 1, dtype=np.int32)]
    tok_off = np.concatenate([[0], np.cumsum([len(t) for t in reqs])]).astype(np.int64)
    blk_off = np.concatenate([[0], np.cumsum([len(t) // B for t in reqs])]).astype(np.int64)
    total = int(blk_off[-1])
    extra = rng.integers(0, 1 << 62, total).astype(np.uint64)
    ctx = wpp.Context(0)
    dev = torch.device("cuda", 0)
    tokens = torch.from_numpy(np.concatenate(reqs)).to(dev)
    for ek in (None, extra):
        ekd = None if ek is None else torch.from_numpy(ek.view(np.int64)).to(dev)
        out = wpp.wpp_hash_blocks(ctx, tokens, torch.from_numpy(tok_off).to(dev), torch.from_numpy(blk_off).to(dev),
                                  B, salt=77, extra_keys=ekd)
        got = out.cpu().numpy().view(np.uint64)
        for i, t in enumerate(reqs):
            e = None if ek is None else ek[blk_off[i]:blk_off[i + 1]].tolist()
            assert got[blk_off[i]:blk_off[i + 1]].tolist() == O.chained_hashes(t.tolist(), B, 77, e)
