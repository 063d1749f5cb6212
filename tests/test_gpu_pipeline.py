"""The upstream steps and the kernels in a row on the GPU: token blocks are hashed (wpp_hash_blocks), the hint index
gives each request's reused prefix, wpp_plan_waves cuts the uncached suffixes into waves, and every wave goes
through wpp_plan_tiles, wpp_kv_append and wpp_prefill_attention_varlen.  Whatever chunking the planner chose, the
pools must end up bit-identical to, and the outputs within tolerance of, the oracle's one-shot result (chunked
prefill over a cached prefix equals full-sequence causal attention, for any chunk split)."""
import copy

import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests import gpu_harness as H
from tests.helpers import bits, cpu_inputs, f64, run_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,b_min,lanes", [(1024, 256, 4), (512, 512, 2), (2048, 128, 8)])
def test_waves_planned_from_hashed_prefixes_equal_the_one_shot_result(M, b_min, lanes):
    B, Hq, Hkv, d = 64, 8, 2, 128
    rng = np.random.default_rng(M + lanes)
    shared_blocks = 6
    # token ids: four requests start with the same 6 blocks, two do not; suffix lengths are ragged
    common = rng.integers(0, 30000, shared_blocks * B).astype(np.int32)
    suffix = [700, 64, 1300, 333, 900, 17]
    sharer = [True, True, False, True, True, False]
    private_prefix = [0, 0, 128, 0, 0, 0]                      # request 2 has two cached blocks of its own
    toks = []
    for i in range(6):
        head = common if sharer[i] else rng.integers(0, 30000, private_prefix[i]).astype(np.int32)
        toks.append(np.concatenate([head, rng.integers(0, 30000, suffix[i]).astype(np.int32)]))

    # ---- prefix hints: what is cached so far is the common prefix and request 2's own blocks
    ctx = H.ctx()
    dev = torch.device("cuda")
    tok_off = np.concatenate([[0], np.cumsum([len(t) for t in toks])]).astype(np.int64)
    blk_off = np.concatenate([[0], np.cumsum([len(t) // B for t in toks])]).astype(np.int64)
    hashes = wpp.wpp_hash_blocks(ctx, torch.from_numpy(np.concatenate(toks)).to(dev), torch.from_numpy(tok_off).to(dev),
                                 torch.from_numpy(blk_off).to(dev), B, salt=5).cpu().numpy().view(np.uint64)
    idx = wpp.HintIndex()
    idx.add(0, wpp.wpp_hash_blocks_host(common, B, salt=5))
    idx.add(0, hashes[blk_off[2]:blk_off[2] + private_prefix[2] // B])
    cached = [idx.probe(0, hashes[blk_off[i]:blk_off[i + 1]])[0] * B for i in range(6)]
    assert cached == [shared_blocks * B if s else p for s, p in zip(sharer, private_prefix)]

    # ---- the one-shot reference: every request's whole suffix as one chunk over its cached prefix
    w_all = W.make_workload("pipeline", 3, np.random.default_rng(3), cached, suffix, Hq, Hkv, d, B,
                            shared_tokens=shared_blocks * B, sharers=np.array(sharer))
    inp = cpu_inputs(w_all)
    kp_ref, vp_ref, ref, _ = run_oracle(w_all, inp)
    devin = H.device_inputs(w_all, inp)
    row0 = np.concatenate([[0], np.cumsum(suffix)])

    # ---- waves
    cfg = wpp.WaveConfig(2, 2, B, lanes, M, b_min)
    st = wpp.WaveState(len(wpp.wpp_wave_ladder(cfg)) - 1, 0, 0, 0)
    done = np.zeros(6, dtype=np.int64)
    got = np.full(ref.shape, np.nan)
    inflight, waves = [], 0
    while done.sum() < sum(suffix):
        chunks, info = wpp.wpp_plan_waves(cfg, st, (np.array(suffix) - done).tolist(), [c for wv in inflight for c in wv])
        assert info.wave_tokens > 0 and info.wave_tokens <= info.budget and info.lanes <= lanes
        rows = np.concatenate([np.arange(row0[i] + done[i], row0[i] + done[i] + chunks[i]) for i in range(6)])
        w = copy.copy(w_all)
        w.prefix_lens = (np.array(cached) + done).astype(np.int32)
        w.chunk_lens = chunks.astype(np.int32)
        sel = torch.from_numpy(rows).to(dev)
        part = dict(q=devin["q"][sel].contiguous(), k_new=devin["k_new"][sel].contiguous(),
                    v_new=devin["v_new"][sel].contiguous(), k_pool=devin["k_pool"], v_pool=devin["v_pool"])
        res = H.run_wave(w, part)
        assert res["status"] == 0
        got[rows] = f64(res["out"])
        done += chunks
        inflight = (inflight + [[int(c) for c in chunks if c]])[-4:]
        waves += 1
    assert waves >= 2
    assert np.array_equal(bits(devin["k_pool"]), kp_ref) and np.array_equal(bits(devin["v_pool"]), vp_ref)
    H.assert_close(got, ref, "waves from the planner")
