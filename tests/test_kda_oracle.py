"""Pins for the oracle of the recurrent-state layer (Section 3.1's KDA update, Section 3.2's snapshots): a worked
example done by hand, special cases with closed forms, and the chunk-parallel closed form solved with a library
triangular solve - each would fail for a dropped term, a wrong sign, a transposed operand or a decay applied on the
wrong side of the delta rule."""
import numpy as np

from oracle import kda as O


def _rand(rng, T, H, dk, dv, unit_k=False):
    q = rng.standard_normal((T, H, dk))
    k = rng.standard_normal((T, H, dk))
    if unit_k:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((T, H, dv))
    alpha = rng.uniform(0.3, 1.0, (T, H, dk))
    beta = rng.uniform(0.0, 1.0, (T, H))
    return q, k, v, alpha, beta


def _run(q, k, v, alpha, beta, S0=None, **kw):
    T, H, dk = q.shape
    dv = v.shape[2]
    pool = np.zeros((2, H, dk, dv))
    if S0 is not None:
        pool[0] = S0
    o = O.kda_chunk(q, k, v, alpha, beta, [T], pool, [0 if S0 is not None else -1], [1], **kw)
    return o, pool[1]


def test_worked_example_by_hand():
    # d_k = 2, d_v = 1.  Token 1: S0 = (1, 2)^T, alpha = (1/2, 1/4) -> D = (1/2, 1/2)^T; k = (1, 0), k^T D = 1/2;
    # S1 = D - 1/2 * k * 1/2 + 1/2 * k * 3 = (1.75, 0.5)^T; o1 = S1^T (1, 1) = 2.25.
    # Token 2: alpha = 1, k = (0.6, 0.8), beta = 1, v = 2: k^T S1 = 1.45; S2 = S1 + k (2 - 1.45) = (2.08, 0.94)^T;
    # o2 = S2^T (1, 0) = 2.08 (and k^T S2 = 2 = v, the delta rule's retrieval property).
    S0 = np.array([[[1.0], [2.0]]])
    q = np.array([[[1.0, 1.0]], [[1.0, 0.0]]])
    k = np.array([[[1.0, 0.0]], [[0.6, 0.8]]])
    v = np.array([[[3.0]], [[2.0]]])
    alpha = np.array([[[0.5, 0.25]], [[1.0, 1.0]]])
    beta = np.array([[0.5], [1.0]])
    o, S = _run(q, k, v, alpha, beta, S0)
    assert np.allclose(o[:, 0, 0], [2.25, 2.08], rtol=0, atol=1e-14)
    assert np.allclose(S[0, :, 0], [2.08, 0.94], rtol=0, atol=1e-14)


def test_delta_rule_retrieves_the_value_just_written():
    # alpha = 1, beta = 1, |k| = 1: S_t^T k_t = S'^T k - (k^T k) S'^T k + (k^T k) v = v_t
    rng = np.random.default_rng(0)
    T, H, dk, dv = 9, 2, 8, 5
    q, k, v, alpha, beta = _rand(rng, T, H, dk, dv, unit_k=True)
    S0 = rng.standard_normal((H, dk, dv))
    for t in range(1, T + 1):
        o, _ = _run(np.concatenate([q[:t - 1], k[t - 1:t]]), k[:t], v[:t], np.ones((t, H, dk)), np.ones((t, H)), S0)
        assert np.allclose(o[t - 1], v[t - 1], atol=1e-12)


def test_beta_zero_is_pure_decay():
    # S_t = Diag(prod alpha) S_0, o_t = S_0^T (Gamma_t * q_t)
    rng = np.random.default_rng(1)
    T, H, dk, dv = 7, 3, 6, 4
    q, k, v, alpha, _ = _rand(rng, T, H, dk, dv)
    S0 = rng.standard_normal((H, dk, dv))
    o, S = _run(q, k, v, alpha, np.zeros((T, H)), S0)
    gamma = np.cumprod(alpha, axis=0)
    assert np.allclose(S, gamma[-1][:, :, None] * S0, atol=1e-13)
    assert np.allclose(o, np.einsum("hkv,thk->thv", S0, gamma * q), atol=1e-12)


def test_orthonormal_keys_without_decay_are_causal_linear_attention():
    # keys orthonormal, alpha = 1, S_0 = 0: k_t^T S_{t-1} = 0, so S_t = sum beta_s k_s v_s^T and
    # O = tril(Q K^T) diag(beta) V  (one library matmul per head)
    rng = np.random.default_rng(2)
    T, H, dk, dv = 6, 2, 8, 3
    q, _, v, _, beta = _rand(rng, T, H, dk, dv)
    k = np.stack([np.linalg.qr(rng.standard_normal((dk, dk)))[0][:T] for _ in range(H)], axis=1)
    o, S = _run(q, k, v, np.ones((T, H, dk)), beta)
    for h in range(H):
        A = np.tril(q[:, h] @ k[:, h].T)
        assert np.allclose(o[:, h], A @ (beta[:, h, None] * v[:, h]), atol=1e-12)
        assert np.allclose(S[h], k[:, h].T @ (beta[:, h, None] * v[:, h]), atol=1e-12)


def test_chunk_parallel_closed_form_with_a_triangular_solve():
    # With Gamma_t = prod_{s<=t} alpha_s:  S_t = Diag(Gamma_t) S_0 + sum_{s<=t} Diag(Gamma_t / Gamma_s) k_s u_s^T where
    # (I + A) U = diag(beta) (V - (K*Gamma) S_0),  A[t,s] = beta_t ((k_t*Gamma_t) . (k_s/Gamma_s)) for s < t, and
    # O = (Q*Gamma) S_0 + tril((Q*Gamma)(K/Gamma)^T) U.  The unknowns come from numpy's linear solver.
    rng = np.random.default_rng(3)
    T, H, dk, dv = 24, 2, 16, 12
    q, k, v, alpha, beta = _rand(rng, T, H, dk, dv)
    S0 = rng.standard_normal((H, dk, dv))
    o, S = _run(q, k, v, alpha, beta, S0)
    for h in range(H):
        G = np.cumprod(alpha[:, h], axis=0)
        Kt, Kh, Qt = k[:, h] * G, k[:, h] / G, q[:, h] * G
        A = np.tril(beta[:, h, None] * (Kt @ Kh.T), -1)
        U = np.linalg.solve(np.eye(T) + A, beta[:, h, None] * (v[:, h] - Kt @ S0[h]))
        assert np.allclose(o[:, h], Qt @ S0[h] + np.tril(Qt @ Kh.T) @ U, atol=1e-10)
        assert np.allclose(S[h], G[-1][:, None] * S0[h] + (Kh * G[-1]).T @ U, atol=1e-10)


def test_resuming_from_a_snapshot_equals_running_through():
    # Section 3.2: the state after exactly r tokens is what a recurrent layer resumes from
    rng = np.random.default_rng(4)
    H, dk, dv = 2, 8, 8
    lens, prefix, interval = [37, 5, 64], [11, 0, 128], 16
    T = sum(lens)
    q, k, v, alpha, beta = _rand(rng, T, H, dk, dv, unit_k=True)
    pool = rng.standard_normal((16, H, dk, dv))
    start = pool.copy()
    snaps = np.full((3, 5), -1)
    snaps[0, :3] = [4, 5, 6]            # positions 16, 32, 48 of request 0 (prefix 11, chunk 37 -> ends at 48)
    snaps[2, :4] = [7, -1, 9, 10]       # positions 144, (160 skipped), 176, 192 of request 2
    o = O.kda_chunk(q, k, v, alpha, beta, lens, pool, [0, -1, 1], [2, 3, -1], prefix, interval, snaps)
    assert np.array_equal(pool[:2], start[:2]) and np.array_equal(pool[8], start[8])     # inputs and skipped slots untouched
    assert np.array_equal(pool[6], pool[2])                                               # boundary at the chunk end
    assert np.array_equal(pool[10], _rerun(q, k, v, alpha, beta, 42, 64, start[1])[1])
    # request 0 resumed from its snapshot at position 32 (21 tokens in): the remaining 16 outputs are the same
    o2, S2 = _rerun(q, k, v, alpha, beta, 21, 16, pool[5])
    assert np.allclose(o2, o[21:37], atol=1e-12) and np.allclose(S2, pool[2], atol=1e-12)
    # request 1 started from the zero state
    o1, S1 = _rerun(q, k, v, alpha, beta, 37, 5, None)
    assert np.allclose(o1, o[37:42], atol=1e-14) and np.allclose(S1, pool[3], atol=1e-14)


def _rerun(q, k, v, alpha, beta, row, n, S0):
    sl = slice(row, row + n)
    return _run(q[sl], k[sl], v[sl], alpha[sl], beta[sl], S0)


def test_empty_chunks_copy_the_state_and_snapshot_size():
    rng = np.random.default_rng(5)
    pool = rng.standard_normal((3, 1, 4, 4))
    z = np.zeros((0, 1, 4))
    o = O.kda_chunk(z, z, z, z, np.zeros((0, 1)), [0, 0], pool, [0, -1], [1, 2])
    assert o.shape == (0, 1, 4) and np.array_equal(pool[1], pool[0]) and not pool[2].any()
    # one fp32 checkpoint of 32 heads of 128 x 128 is 2 MiB per linear layer
    assert O.snapshot_bytes(4, 32, 128, 128) == 2 << 20 and O.snapshot_bytes(2, 8, 64, 128, layers=3) == 393216
