"""Pins for the fp64 oracle: everything here checks it against something other than itself.

The paper prints no worked attention example, so the pins are brute force on tiny
inputs, invariants that the setting fixes (chunking, paging, sharing), closed forms
and a library special case (torch SDPA in fp64).
"""
import math

import numpy as np
import pytest
import torch

import oracle
import wpp_workloads as W
from tests.helpers import bits, cpu_inputs, f64, from_bits, run_oracle


# ----------------------------------------------------------------- I1 brute force
@pytest.mark.parametrize("P,C,Hq,Hkv,d,B", [
    ([0], [1], 1, 1, 8, 1),
    ([5], [7], 2, 1, 8, 2),
    ([16], [16], 4, 2, 16, 4),
    ([0, 3, 33], [9, 1, 31], 4, 1, 16, 16),
    ([7, 0], [25, 40], 8, 2, 32, 16),
    ([48], [16], 4, 4, 64, 16),
])
def test_I1_matches_brute_dense(P, C, Hq, Hkv, d, B):
    w = W.custom_workload(P, C, Hq, Hkv, d, B, seed=11)
    inp = cpu_inputs(w)
    kp, vp, out, lse = run_oracle(w, inp)
    bo, bl = oracle.brute_dense(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens)
    np.testing.assert_allclose(out, bo, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, bl, rtol=0, atol=1e-12)


def test_I1_explicit_scale_matches_brute():
    w = W.custom_workload([6], [10], 2, 2, 16, 4, seed=12)
    inp = cpu_inputs(w)
    kp, vp, out, lse = run_oracle(w, inp, sm_scale=0.37)
    bo, bl = oracle.brute_dense(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, sm_scale=0.37)
    np.testing.assert_allclose(out, bo, atol=1e-12)
    np.testing.assert_allclose(lse, bl, atol=1e-12)


# ------------------------------------------------- I2 / I4 chunking does not matter
def _run_in_chunks(w_full, splits):
    """Process one request's tokens [0, n) in successive calls of the given chunk lengths."""
    inp = cpu_inputs(w_full)
    kp, vp = bits(inp["k_pool"]).copy(), bits(inp["v_pool"]).copy()
    n = int(w_full.chunk_lens[0])
    outs, lses, start = [], [], 0
    for c in splits:
        sl = slice(start, start + c)
        kp, vp = oracle.oracle_append(inp["k_new"][sl], inp["v_new"][sl], kp, vp, w_full.block_tables,
                                      [start], [c])
        o, l = oracle.oracle_attention(inp["q"][sl], kp, vp, w_full.block_tables, [start], [c])
        outs.append(o)
        lses.append(l)
        start += c
    assert start == n
    return np.concatenate(outs), np.concatenate(lses), kp, vp


@pytest.mark.parametrize("splits", [[37], [20, 17], [1, 35, 1], [16, 16, 5], [5, 4, 3, 25]])
def test_I2_I4_any_chunk_split_equals_one_shot(splits):
    w = W.custom_workload([0], [37], 4, 2, 16, 4, seed=21)
    kp1, vp1, out1, lse1 = run_oracle(w)
    out, lse, kp, vp = _run_in_chunks(w, splits)
    # identical summation order => identical bits
    assert np.array_equal(out, out1) and np.array_equal(lse, lse1)
    assert np.array_equal(kp, kp1) and np.array_equal(vp, vp1)


def test_I2_prefix_reuse_equals_recompute():
    """A request whose first p tokens are already cached gives the rows of full recomputation."""
    n, p = 45, 29            # p deliberately not a page multiple
    w = W.custom_workload([0], [n], 2, 1, 8, 4, seed=22)
    inp = cpu_inputs(w)
    _, _, out_full, _ = run_oracle(w, inp)
    kp, vp = oracle.oracle_append(inp["k_new"][:p], inp["v_new"][:p], inp["k_pool"], inp["v_pool"],
                                  w.block_tables, [0], [p])
    kp, vp = oracle.oracle_append(inp["k_new"][p:], inp["v_new"][p:], kp, vp, w.block_tables, [p], [n - p])
    out, _ = oracle.oracle_attention(inp["q"][p:], kp, vp, w.block_tables, [p], [n - p])
    assert np.array_equal(out, out_full[p:])


# ------------------------------------------------------- I3 shared == private pages
def test_I3_shared_pages_equal_private_copies():
    B, d, Hkv, Hq = 4, 8, 2, 4
    shared_tokens = 12
    R = 5
    P = [12, 15, 12, 19, 13]
    C = [3, 6, 1, 4, 9]
    rng = np.random.default_rng(31)
    ws = W.make_workload("shared", 31, rng, P, C, Hq, Hkv, d, B, shared_tokens=shared_tokens,
                         sharers=[True] * R, spare_pages=40)
    inp = cpu_inputs(ws)
    # every table starts with the same three physical pages
    assert all(np.array_equal(ws.block_tables[i, :3], ws.block_tables[0, :3]) for i in range(R))
    _, _, out_s, lse_s = run_oracle(ws, inp)
    # private copies: give each request its own copy of the shared pages among the spare ones
    kp, vp = bits(inp["k_pool"]).copy(), bits(inp["v_pool"]).copy()
    bt = ws.block_tables.copy()
    used = set(bt[bt >= 0].tolist())
    free = [p for p in range(ws.num_pages) if p not in used]
    for i in range(1, R):
        for j in range(shared_tokens // B):
            new = free.pop()
            kp[new], vp[new] = kp[bt[0, j]], vp[bt[0, j]]
            bt[i, j] = new
    kp2, vp2 = oracle.oracle_append(inp["k_new"], inp["v_new"], kp, vp, bt, P, C)
    out_p, lse_p = oracle.oracle_attention(inp["q"], kp2, vp2, bt, P, C)
    assert np.array_equal(out_s, out_p) and np.array_equal(lse_s, lse_p)


# ------------------------------------------------------------------ I5 closed forms
def _tiny(seed=41, P=9, C=6, Hq=4, Hkv=2, d=8, B=4):
    w = W.custom_workload([P], [C], Hq, Hkv, d, B, seed=seed)
    return w, cpu_inputs(w)


def test_I5_single_key_returns_v0_exactly():
    w = W.custom_workload([0], [1], 4, 2, 8, 4, seed=42)
    inp = cpu_inputs(w)
    _, _, out, lse = run_oracle(w, inp)
    v0 = f64(inp["v_new"])[0]                       # [Hkv, d]
    for h in range(4):
        assert np.array_equal(out[0, h], v0[h // 2])
    k0, q0 = f64(inp["k_new"])[0], f64(inp["q"])[0]
    for h in range(4):
        assert lse[0, h] == pytest.approx(float(q0[h] @ k0[h // 2]) / math.sqrt(8), abs=1e-13)


def test_I5_zero_query_gives_running_mean_of_v():
    w, inp = _tiny()
    inp["q"] = torch.zeros_like(inp["q"])
    kp, vp, out, lse = run_oracle(w, inp)
    P, C = 9, 6
    V = oracle.gather_contiguous(vp, w.block_tables[0], P + C)       # [n, Hkv, d]
    for t in range(C):
        for h in range(4):
            np.testing.assert_allclose(out[t, h], V[:P + t + 1, h // 2].mean(axis=0), atol=1e-14)
            assert lse[t, h] == pytest.approx(math.log(P + t + 1), abs=1e-14)


def test_I5_constant_v_gives_constant_output():
    w, inp = _tiny(seed=43)
    c = 0.8125
    inp["v_new"] = torch.full_like(inp["v_new"], c)
    inp["v_pool"] = torch.full_like(inp["v_pool"], c)
    _, _, out, _ = run_oracle(w, inp)
    np.testing.assert_allclose(out, c, atol=1e-15)


def test_I5_shift_invariance_exact_on_dyadic_inputs():
    """Adding one vector u to every key shifts each row's scores by a constant: O is unchanged, lse moves by q.u/sqrt(d).
    Keys are quantised so that k + u is exactly representable in bf16."""
    w, inp = _tiny(seed=45)
    # quantise keys to multiples of 1/4 in [-4, 4] so that k + u is exact in bf16
    for name in ("k_new", "k_pool"):
        inp[name] = (torch.round(inp[name].double() * 4) / 4).clamp(-4, 4).to(torch.bfloat16)
    u = torch.tensor([0.5, -1.0, 2.0, 0.25, -0.5, 1.0, 0.0, -2.0], dtype=torch.float64)
    _, _, out0, lse0 = run_oracle(w, inp)
    inp2 = dict(inp)
    for name in ("k_new", "k_pool"):
        shifted = inp[name].double() + u
        inp2[name] = shifted.to(torch.bfloat16)
        assert torch.equal(inp2[name].double(), shifted)
    _, _, out1, lse1 = run_oracle(w, inp2)
    np.testing.assert_allclose(out1, out0, atol=1e-13)
    shift = (f64(inp["q"]) @ u.numpy()) / math.sqrt(8)
    np.testing.assert_allclose(lse1 - lse0, shift, atol=1e-12)


def test_I5_v_scaling_by_power_of_two_is_exact():
    w, inp = _tiny(seed=46)
    _, _, out0, lse0 = run_oracle(w, inp)
    inp2 = dict(inp)
    inp2["v_new"] = inp["v_new"] * 8
    inp2["v_pool"] = inp["v_pool"] * 8
    _, _, out1, lse1 = run_oracle(w, inp2)
    assert np.array_equal(out1, out0 * 8) and np.array_equal(lse1, lse0)


def test_I5_gqa_equals_mha_with_duplicated_kv_heads():
    w, inp = _tiny(seed=47, Hq=4, Hkv=2)
    kp, vp, out0, lse0 = run_oracle(w, inp)
    # MHA problem with Hkv' = Hq: kv head h' = h holds a copy of kv head h // G
    idx = torch.tensor([0, 0, 1, 1])
    kp_m = from_bits(kp)[:, idx].contiguous()
    vp_m = from_bits(vp)[:, idx].contiguous()
    out1, lse1 = oracle.oracle_attention(inp["q"], kp_m, vp_m, w.block_tables, w.prefix_lens, w.chunk_lens)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


def test_I5_head_mapping_is_consecutive_groups():
    """kv_head = q_head // G: zero one kv head's V and see exactly its group's outputs vanish."""
    w, inp = _tiny(seed=48, Hq=6, Hkv=3)
    inp["v_new"][:, 1] = 0
    inp["v_pool"][:, 1] = 0
    _, _, out, _ = run_oracle(w, inp)
    assert np.all(out[:, 2:4] == 0) and np.all(np.abs(out[:, [0, 1, 4, 5]]).sum(axis=-1) > 0)


# ------------------------------------------------------------ I6 library special case
@pytest.mark.parametrize("P,C", [(0, 24), (19, 13), (64, 1)])
def test_I6_matches_torch_sdpa_fp64(P, C):
    Hq, Hkv, d, B = 4, 2, 16, 8
    w = W.custom_workload([P], [C], Hq, Hkv, d, B, seed=51)
    inp = cpu_inputs(w)
    kp, vp, out, _ = run_oracle(w, inp)
    n = P + C
    K = torch.from_numpy(oracle.gather_contiguous(kp, w.block_tables[0], n))     # [n, Hkv, d]
    V = torch.from_numpy(oracle.gather_contiguous(vp, w.block_tables[0], n))
    K = K.repeat_interleave(Hq // Hkv, dim=1).permute(1, 0, 2)[None]            # [1, Hq, n, d]
    V = V.repeat_interleave(Hq // Hkv, dim=1).permute(1, 0, 2)[None]
    Q = inp["q"].double().permute(1, 0, 2)[None]                                # [1, Hq, C, d]
    mask = torch.arange(n)[None, :] <= (P + torch.arange(C))[:, None]           # bottom-right aligned
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    if P == 0:   # torch's own causal flag is top-left aligned: usable only for a square problem
        ref2 = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True)
        np.testing.assert_allclose(out, ref2[0].permute(1, 0, 2).numpy(), atol=1e-12)


# ----------------------------------------------------------------- I7 page permutation
def test_I7_physical_page_permutation_changes_nothing():
    w = W.custom_workload([10, 0, 21], [6, 9, 3], 4, 2, 8, 4, seed=61, spare_pages=5)
    inp = cpu_inputs(w)
    _, _, out0, lse0 = run_oracle(w, inp)
    perm = np.random.default_rng(62).permutation(w.num_pages)          # old id -> new id
    kp = torch.empty_like(inp["k_pool"])
    vp = torch.empty_like(inp["v_pool"])
    kp[perm] = inp["k_pool"]
    vp[perm] = inp["v_pool"]
    bt = np.where(w.block_tables >= 0, perm[np.maximum(w.block_tables, 0)], -1).astype(np.int32)
    kp2, vp2 = oracle.oracle_append(inp["k_new"], inp["v_new"], kp, vp, bt, w.prefix_lens, w.chunk_lens)
    out1, lse1 = oracle.oracle_attention(inp["q"], kp2, vp2, bt, w.prefix_lens, w.chunk_lens)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


# ------------------------------------------------------------------ I8 LSE merge identity
@pytest.mark.parametrize("cuts", [[5], [1, 2], [3, 9, 14], [2, 4, 6, 8, 10, 12]])
def test_I8_merging_key_partitions_reproduces_full_softmax(cuts):
    w = W.custom_workload([11], [5], 2, 1, 8, 4, seed=71)
    inp = cpu_inputs(w)
    kp, vp, out, lse = run_oracle(w, inp)
    n_all = 16
    K = oracle.gather_contiguous(kp, w.block_tables[0], n_all)[:, 0]
    V = oracle.gather_contiguous(vp, w.block_tables[0], n_all)[:, 0]
    q = f64(inp["q"])
    for t in range(5):
        n = 11 + t + 1
        edges = [0] + [c for c in cuts if c < n] + [n]
        for h in range(2):
            parts_o, parts_l = [], []
            for a, b in zip(edges[:-1], edges[1:]):
                s = (K[a:b] @ q[t, h]) / math.sqrt(8)
                m = s.max()
                wgt = np.exp(s - m)
                parts_o.append((wgt[:, None] * V[a:b]).sum(0) / wgt.sum())
                parts_l.append(m + math.log(wgt.sum()))
            o, l = oracle.merge_partials(np.array(parts_o), np.array(parts_l))
            np.testing.assert_allclose(o, out[t, h], atol=1e-13)
            assert l == pytest.approx(lse[t, h], abs=1e-13)


def test_I8_merge_ignores_empty_partition():
    o, l = oracle.merge_partials(np.array([[1.0, 2.0], [0.0, 0.0]]), np.array([0.3, -np.inf]))
    np.testing.assert_allclose(o, [1.0, 2.0])
    assert l == pytest.approx(0.3)


# --------------------------------------------------------------------- I9 append round trip
def test_I9_append_round_trip_and_untouched_bytes():
    w = W.custom_workload([10, 0, 21, 5], [6, 9, 3, 0], 4, 2, 8, 4, seed=81, spare_pages=5)
    inp = cpu_inputs(w)
    # poison patterns must survive bit for bit: NaN payloads, -0.0, Inf
    kn = bits(inp["k_new"]).copy()
    kn[0, 0, :4] = [0x7FC1, 0x8000, 0xFF80, 0xFFFF]
    inp["k_new"] = from_bits(kn)
    kp0, vp0 = bits(inp["k_pool"]), bits(inp["v_pool"])
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"],
                                  w.block_tables, w.prefix_lens, w.chunk_lens)
    touched = np.zeros(kp.shape[:1] + kp.shape[2:3], dtype=bool)       # [page, slot]
    off = 0
    for i in range(w.num_requests):
        P, C = int(w.prefix_lens[i]), int(w.chunk_lens[i])
        for t in range(C):
            pos = P + t
            page, slot = int(w.block_tables[i, pos // 4]), pos % 4
            assert np.array_equal(kp[page, :, slot], kn[off + t])
            assert np.array_equal(vp[page, :, slot], bits(inp["v_new"])[off + t])
            touched[page, slot] = True
        off += C
    assert touched.sum() == w.total_new_tokens
    untouched = ~touched[:, None, :, None] & np.ones(kp.shape, dtype=bool)
    assert np.array_equal(kp[untouched], kp0[untouched]) and np.array_equal(vp[untouched], vp0[untouched])


def test_append_rejects_bad_page_id():
    w = W.custom_workload([0], [5], 2, 1, 8, 4, seed=82)
    inp = cpu_inputs(w)
    bt = w.block_tables.copy()
    bt[0, 1] = w.num_pages
    with pytest.raises(ValueError):
        oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"], bt, [0], [5])


# --------------------------------------------------- stale slots / unreferenced pages (Q9)
def test_stale_slots_and_unused_pages_do_not_influence_the_result():
    w = W.custom_workload([9, 2], [6, 3], 4, 2, 8, 4, seed=91, spare_pages=4)
    inp = cpu_inputs(w)
    _, _, out0, lse0 = run_oracle(w, inp)
    kp, vp = bits(inp["k_pool"]).copy(), bits(inp["v_pool"]).copy()
    live = np.zeros((w.num_pages, 4), dtype=bool)
    for i in range(2):
        n_prefix = int(w.prefix_lens[i])
        for pos in range(n_prefix):
            live[w.block_tables[i, pos // 4], pos % 4] = True
    dead = ~live
    kp[np.broadcast_to(dead[:, None, :, None], kp.shape)] = 0x7FC0        # NaN everywhere not yet written
    vp[np.broadcast_to(dead[:, None, :, None], vp.shape)] = 0xFFFF
    inp2 = dict(inp, k_pool=from_bits(kp), v_pool=from_bits(vp))
    _, _, out1, lse1 = run_oracle(w, inp2)
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


# ------------------------------------------------------------- probes for mask off-by-one
def test_probe_next_key_must_not_leak_and_diagonal_must_count():
    """Keys crafted as beta*q: the row's own key must dominate, the next row's key must be invisible."""
    P, C, d = 6, 5, 8
    w = W.custom_workload([P], [C], 1, 1, d, 4, seed=101)
    inp = cpu_inputs(w)
    q = inp["q"].double()
    inp["k_new"] = (q * 16).to(torch.bfloat16)                 # K[P+t] = 16 q_t  (diagonal dominates)
    kp, vp, out, _ = run_oracle(w, inp)
    V = oracle.gather_contiguous(vp, w.block_tables[0], P + C)[:, 0]
    qn = (q[:, 0] ** 2).sum(-1)
    for t in range(C):
        if qn[t] > 2.0:                                         # peaked enough: output ~ V[P+t]
            assert np.abs(out[t, 0] - V[P + t]).max() < 0.25
    bo, _ = oracle.brute_dense(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens)
    np.testing.assert_allclose(out, bo, atol=1e-12)


# ------------------------------------------------------------------------- golden regression
def test_golden_cfg1_rows_are_reproduced():
    """Stored by tests/golden/make_golden.py (which calls only the oracle): guards against drift."""
    import json
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "cfg1_oracle_rows.json")
    g = json.load(open(path))
    w = W.cfg1()
    inp = cpu_inputs(w)
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"],
                                  w.block_tables, w.prefix_lens, w.chunk_lens)
    units = np.array(g["units"], dtype=np.int32)
    out, lse = oracle.oracle_attention_units(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, units)
    exp_out = np.array([[float.fromhex(x) for x in row] for row in g["out_hex"]])
    exp_lse = np.array([float.fromhex(x) for x in g["lse_hex"]])
    np.testing.assert_allclose(out, exp_out, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse, exp_lse, rtol=0, atol=1e-13)


def test_units_entry_point_equals_full_run():
    w = W.custom_workload([7, 0], [5, 8], 4, 2, 8, 4, seed=111)
    inp = cpu_inputs(w)
    kp, vp, out, lse = run_oracle(w, inp)
    units = [(0, 0, 0), (0, 4, 3), (1, 7, 2), (1, 0, 1)]
    o, l = oracle.oracle_attention_units(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens, units)
    off = w.q_offsets
    for k, (i, t, h) in enumerate(units):
        assert np.array_equal(o[k], out[off[i] + t, h]) and l[k] == lse[off[i] + t, h]
