"""Every output row of the full-size configurations, checked against closed forms.

A sampled comparison with the oracle sees a few per cent of the work tiles.  The checks here cover EVERY (row, head)
of a wave at the size the benchmark times, using inputs for which the result is known without running anything:

* zero queries: every score is 0, so every visible key has probability exactly 1 before normalisation, the row sum
  is the integer n = P_i + t + 1 (exact in fp32 up to 2^24) and lse = ln n.  One dropped, doubled or leaked
  128-key step moves lse by at least ln(1 + 128/n) > 9e-4 at n = 139,264, where the bf16 output could not show it.
  Bound on the kernel's error, from its arithmetic: lse = (m + log2f(l)) * ln2 with m = 0; log2f is within 1 ulp of
  a value below 17.1 (2^-19 = 1.9e-6), times ln2 = 1.3e-6, plus the rounding of the product (half an ulp of 11.9 =
  4.8e-7) and of the constant (11.9 * 2^-24 = 7e-7): 2.5e-6.  With split tiles every part carries that error, the
  weights exp2f(lse_s - max) add 2 ulp (2.4e-7, relative) and the final log2f of a number in [1, 64] one more ulp
  (4.8e-7): below 6e-6 in all.  The test allows 1e-5.
  The output is then the running mean of V, which the oracle (pinned to that closed form on the CPU) supplies on
  sampled units.
* constant values, V = 1.5 everywhere: the output is 1.5 * sum(bf16(p_j)) / sum(p_j).  Rounding a probability to
  bf16 (8 significant bits) moves it by at most 2^-8 relatively, so the quotient lies within 2^-8 of 1 (fp32
  accumulation adds far less), the result within 0.0059 of 1.5, and the rounded output is 1.5 or one of its two bf16
  neighbours (0.0078 apart).  A neighbour only appears on a row that one key dominates (the rounding errors of many
  comparable probabilities cancel), so nearly every element must be 1.5 bit for bit and no element may be further
  than one step away.  A step counted in the row sum but not in the product (or the other way round), or a wrong
  rescale, breaks it.
* crafted keys (mask probes): K[P_i + t] = 16 q_t makes row t's own key dominate (its output must be V[P_i + t]; a
  dropped diagonal shows), and in a second run K[P_i + t + 1] = 16 q_t makes the NEXT key dominate, which row t must
  not see (a one-step future leak moves the output by O(1)).  Rows 0, 127, 128, the first page crossing and C - 1 of
  every request, compared with the oracle.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2609_35263_b200 as wpp
import wpp_workloads as W
from tests.helpers import bits, f64
from tests import gpu_harness as H
from tests.test_gpu_fullsize import sample_units, gather_units

pytestmark = pytest.mark.gpu

LSE_TOL = 1e-5
WHOLE_POOL_LIMIT = 6 << 30          # bytes of K + V pool up to which the oracle gets the whole pools


def _cases():
    yield "cfg3", W.cfg3, None
    yield "cfg4_alt", lambda: W.cfg4("alternate"), None
    yield "cfg4_alt_split4", lambda: W.cfg4("alternate"), wpp.PlanOpts(0, 0, 4, 0)
    for C, P in ((64, 0), (64, 131072), (8192, 0), (8192, 131072)):
        yield f"cfg5_C{C}_P{P}", (lambda C=C, P=P: W.cfg5_cell(C, P, num_requests=32)), None


CASES = list(_cases())


def _row_positions(w):
    """n = P_i + t + 1 for every row of the wave (int64 [T], on the device)."""
    C = torch.from_numpy(w.chunk_lens.astype(np.int64)).cuda()
    P = torch.from_numpy(w.prefix_lens.astype(np.int64)).cuda()
    req = torch.repeat_interleave(torch.arange(w.num_requests, device="cuda"), C)
    start = torch.from_numpy(w.q_offsets[:-1]).cuda()
    t = torch.arange(int(C.sum()), device="cuda") - start[req]
    return P[req] + t + 1


class _Oracle:
    """The oracle on sampled units, with the whole pools on the host when they fit and request by request
    (pages gathered through the block table) when they do not."""

    def __init__(self, w, dev):
        self.w = w
        pool_bytes = 2 * dev["k_pool"].numel() * 2
        self.whole = pool_bytes <= WHOLE_POOL_LIMIT
        if self.whole:
            self.k_pool, self.v_pool = dev["k_pool"].cpu(), dev["v_pool"].cpu()
            self.requests = None
        else:
            self.requests = (0, w.num_requests // 2, w.num_requests - 1)
            self.slices = {i: H.request_slice(w, dev, i) for i in self.requests}

    def units(self, n_random, seed):
        return sample_units(self.w, n_random, seed, max_boundary_requests=3, requests=self.requests)

    def attention(self, units, q=None, k_new=None, v_new=None, v_pool=None):
        """Reference for `units` with some inputs replaced (device or CPU tensors of the full wave)."""
        w = self.w
        cpu = lambda t: None if t is None else t.cpu()
        q, k_new, v_new = cpu(q), cpu(k_new), cpu(v_new)
        if self.whole:
            kp, vp = oracle.oracle_append(k_new, v_new, self.k_pool, self.v_pool if v_pool is None else cpu(v_pool),
                                          w.block_tables, w.prefix_lens, w.chunk_lens)
            return oracle.oracle_attention_units(q, kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, units)
        ref = np.empty((len(units), w.head_dim))
        lse = np.empty(len(units))
        for i, sl in self.slices.items():
            r0, r1 = sl["rows"]
            kp, vp = oracle.oracle_append(k_new[r0:r1], v_new[r0:r1], sl["k_pool"], sl["v_pool"], sl["block_tables"],
                                          sl["prefix_lens"], sl["chunk_lens"])
            sel = np.nonzero(units[:, 0] == i)[0]
            u = units[sel].copy()
            u[:, 0] = 0
            ref[sel], lse[sel] = oracle.oracle_attention_units(q[r0:r1], kp, vp, sl["block_tables"], sl["prefix_lens"],
                                                               sl["chunk_lens"], u)
        return ref, lse


def _probe_rows(w, i):
    P, C = int(w.prefix_lens[i]), int(w.chunk_lens[i])
    cross = (-P) % w.page_size
    return sorted(t for t in {0, 127, 128, cross, cross - 1, C - 1} if 0 <= t < C)


@pytest.mark.parametrize("name,make,opts", CASES, ids=[c[0] for c in CASES])
def test_every_row_against_closed_forms(name, make, opts):
    w = make()
    dev = H.device_inputs(w)
    orc = _Oracle(w, dev)                      # host copies are taken before the library touches the pools
    T, Hq, G = w.total_new_tokens, w.num_q_heads, w.num_q_heads // w.num_kv_heads
    n_rows = _row_positions(w)

    # ---- zero queries: lse = ln n on every (row, head); output = running mean of V on sampled units
    q0 = torch.zeros_like(dev["q"])
    res = H.run_wave(w, dict(dev, q=q0), opts=opts)
    assert res["status"] == 0
    want = torch.log(n_rows.double())
    err = (res["lse"].double() - want[:, None]).abs()
    assert not torch.isnan(res["lse"]).any(), "an lse was never written"
    worst = float(err.max())
    assert worst <= LSE_TOL, f"{name}: |lse - ln n| = {worst:.3e} at {np.unravel_index(int(err.argmax()), err.shape)}"
    units = orc.units(300, seed=11)
    ref, ref_lse = orc.attention(units, q=q0, k_new=dev["k_new"], v_new=dev["v_new"])
    got, got_lse = gather_units(w, res, units)
    H.assert_close(got, ref, name + " zero queries")
    del q0, res, err

    # ---- constant values: every output element is 1.5 bit for bit
    v15_new = torch.full_like(dev["v_new"], 1.5)
    v15_pool = torch.full_like(dev["v_pool"], 1.5)
    res = H.run_wave(w, dict(dev, v_new=v15_new, v_pool=v15_pool), opts=opts)
    assert res["status"] == 0
    code = res["out"].view(torch.int16)
    bad = (code - 0x3FC0).abs() > 1              # bf16 codes of 1.5 and its two neighbours: 0x3FBF, 0x3FC0, 0x3FC1
    assert not bool(bad.any()), f"{name}: {int(bad.sum())} output elements are further than one bf16 step from " \
                                f"1.5, first at {np.unravel_index(int(bad.flatten().to(torch.uint8).argmax()), tuple(bad.shape))}"
    off_by_one = int((code != 0x3FC0).sum())
    assert off_by_one <= 1e-4 * code.numel(), f"{name}: {off_by_one} elements one step away from 1.5"
    print(name, "constant V: elements one bf16 step away from 1.5:", off_by_one, "of", code.numel())
    del v15_new, v15_pool, res, bad, code

    # ---- crafted keys at the mask's edge: rows 0, 127, 128, the first page crossing and C - 1 of every request
    reqs = range(w.num_requests) if orc.requests is None else orc.requests
    off = w.q_offsets
    for shift, what in ((0, "own key dominates"), (1, "next key dominates and must stay invisible")):
        k_new = dev["k_new"].clone()
        probe_units = []
        for i in range(w.num_requests):
            C = int(w.chunk_lens[i])
            for t in _probe_rows(w, i):
                if t + shift < C:
                    # KV head g gets 16 x the query of the first query head of its group
                    k_new[off[i] + t + shift] = dev["q"][off[i] + t, ::G] * 16
                if i in reqs:
                    probe_units += [(i, tt, h) for tt in (t - 1, t, t + 1) if 0 <= tt < C for h in range(0, Hq, G)]
                    probe_units += [(i, t, Hq - 1)]
        probe_units = np.array(sorted(set(probe_units)), dtype=np.int32)
        res = H.run_wave(w, dict(dev, k_new=k_new), opts=opts)
        assert res["status"] == 0
        ref, ref_lse = orc.attention(probe_units, q=dev["q"], k_new=k_new, v_new=dev["v_new"])
        got, got_lse = gather_units(w, res, probe_units)
        H.assert_close(got, ref, f"{name}: {what}")
        assert np.abs(got_lse - ref_lse).max() <= 1e-3 * np.maximum(1.0, np.abs(ref_lse)).max()
        if shift == 0:
            # closed form: the probed row returns its own value row
            for i in list(reqs)[:3]:
                for t in _probe_rows(w, i):
                    mine = res["out"][off[i] + t, ::G].double()
                    assert float((mine - dev["v_new"][off[i] + t].double()).abs().max()) <= 2e-2
        assert not torch.isnan(res["out"].float()).any()
        del k_new, res
    torch.cuda.empty_cache()
