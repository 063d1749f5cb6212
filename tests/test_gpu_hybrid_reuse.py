"""Prefix reuse for the recurrent layer end to end on the GPU (Sections 3.2 and 4.3): request A runs a shared prompt
through wpp_kda_chunk with periodic snapshots and publishes the snapshot boundaries in the hint index; request B,
which shares only part of that prompt, finds the dense attention endpoint by galloping, walks back to the deepest
snapshot at or below it, resumes from that slot and must reproduce, from there on, what the oracle computes for
B's whole sequence from the zero state."""
import numpy as np
import pytest
import torch

import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from oracle import kda as O
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu
ATT, REC = 0, 1


def _run(t, rows, H_, state_pool, s_in, s_out, prefix, interval=0, snaps=None):
    dev = torch.device("cuda")
    sel = torch.from_numpy(rows)
    g = {k: t[k][sel].contiguous().to(dev) for k in ("q", "k", "v", "alpha", "beta")}
    i32 = lambda a: None if a is None else torch.tensor(a, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = wpp.wpp_kda_chunk(H.ctx(), g["q"], g["k"], g["v"], g["alpha"], g["beta"],
                            torch.tensor([0, len(rows)], dtype=torch.int64, device=dev), state_pool, i32([s_in]),
                            i32([s_out]), prefix_lens=i32([prefix]), snap_interval=interval,
                            snap_slots=None if snaps is None else i32([snaps]), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.float().cpu().double().numpy()


def test_request_b_resumes_from_the_deepest_usable_snapshot():
    Bsz, H_, interval_blocks = 16, 2, 3                       # 16-token blocks, a snapshot every 3 blocks (48 tokens)
    nA, shared_blocks, nB = 200, 8, 170                       # B shares A's first 8 blocks (128 tokens), then differs
    w = W.kda_workload("hybrid", 31, [nA + nB], H_)
    t = w.tensors()                                           # rows [0, nA): A's tokens; rows [nA, nA + nB): B's own tail
    rng = np.random.default_rng(31)
    tokA = rng.integers(0, 50000, nA).astype(np.int32)
    tokB = np.concatenate([tokA[:shared_blocks * Bsz], rng.integers(0, 50000, nB - shared_blocks * Bsz).astype(np.int32)])
    rowsA = np.arange(nA)
    rowsB = np.concatenate([np.arange(shared_blocks * Bsz), nA + np.arange(nB - shared_blocks * Bsz)])   # B's inputs: A's on the shared part

    # ---- request A: whole prompt from the zero state, snapshots at every third block boundary
    dev = torch.device("cuda")
    n_snaps = nA // (interval_blocks * Bsz)
    pool = torch.zeros(n_snaps + 2, H_, 128, 128, dtype=torch.float32, device=dev)
    _run(t, rowsA, H_, pool, -1, n_snaps, 0, interval_blocks * Bsz, list(range(n_snaps)))
    hA = wpp.wpp_hash_blocks_host(tokA, Bsz)
    idx = wpp.HintIndex()
    idx.add(ATT, hA)
    idx.add(REC, [hA[(j + 1) * interval_blocks - 1] for j in range(n_snaps)])

    # ---- request B: dense endpoint, backward scan, candidate
    hB = wpp.wpp_hash_blocks_host(tokB, Bsz)
    att, _ = idx.probe(ATT, hB)
    rec, probes = idx.probe_recurrent(REC, hB, att)
    assert att == shared_blocks and rec == 6 and probes == 3  # snapshots at 3, 6, 9, ...: 8 -> 7 -> 6
    resume_tokens = min(att, rec) * Bsz
    slot = rec // interval_blocks - 1
    got = _run(t, rowsB[resume_tokens:], H_, pool, slot, n_snaps + 1, resume_tokens)

    # ---- the oracle runs B's whole sequence from the zero state
    f = lambda x: x[torch.from_numpy(rowsB)].double().numpy()
    ref_pool = np.zeros((1, H_, 128, 128))
    ref = O.kda_chunk(f(t["q"]), f(t["k"]), f(t["v"]), f(t["alpha"]), f(t["beta"]), [nB], ref_pool, [-1], [0])
    ref = ref[resume_tokens:]
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-4 * np.abs(ref).max())
    final = pool[n_snaps + 1].double().cpu().numpy()
    assert np.abs(final - ref_pool[0]).max() <= 1e-4 * np.abs(ref_pool[0]).max()
