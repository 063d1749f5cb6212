"""Oracle for the recurrent-state (KDA) layer of a chunk: Section 3.1's simplified single-head update

    S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,        o_t = S_t^T q_t,

taken token by token in fp64, per request and head, resumed from the state after exactly the reused prefix (Section
3.2: a recurrent layer resumes from S_r and nothing else) and snapshotted at the chunk end and at sparse periodic
boundaries (Section 3.2: snapshots only at selected boundaries).

TEST INFRASTRUCTURE ONLY: plain numpy; shares no code with the library's kernel (`wpp_kda_chunk`); only tests,
the smoke check and the CPU-baseline leg of the benchmark import it.

Shapes: S is d_k x d_v; k_t, q_t, alpha_t have d_k entries, v_t and o_t have d_v entries, beta_t is a scalar.
READINGS (the paper gives the update for one head and says nothing else):
  * heads are independent and each has its own state; a batch is ragged like the attention path's (request i owns
    chunk_lens[i] consecutive rows of the packed q/k/v/alpha/beta arrays);
  * no normalisation or scaling of q or k happens inside the operation (the printed update has none): whatever the
    model applies before it is part of the inputs;
  * a periodic snapshot is the state after exactly p tokens of the sequence for every multiple p of the interval
    with prefix < p <= prefix + chunk.
"""
import numpy as np


def kda_step(S, q, k, v, alpha, beta):
    """One token, one head.  S: [d_k, d_v] (modified copy returned), q, k, alpha: [d_k], v: [d_v], beta: scalar."""
    D = alpha[:, None] * S                               # Diag(alpha_t) S_{t-1}
    S_new = D - beta * np.outer(k, k @ D) + beta * np.outer(k, v)
    return S_new, S_new.T @ q


def kda_chunk(q, k, v, alpha, beta, chunk_lens, state_pool, state_in, state_out,
              prefix_lens=None, snap_interval=0, snap_slots=None):
    """The whole ragged batch.

    q, k, alpha : [T, H, d_k]; v : [T, H, d_v]; beta : [T, H]  (any float dtype; computed in fp64)
    state_pool  : float64 [num_slots, H, d_k, d_v], updated in place
    state_in[i] : slot holding S after the reused prefix of request i, or -1 for the zero state
    state_out[i]: slot that receives the state after the chunk, or -1
    snap_slots  : int [num_requests, max_snaps] (or None): slot for the n-th interval boundary inside the chunk, -1 = skip
    Returns o : float64 [T, H, d_v].
    """
    q, k, v = np.asarray(q, np.float64), np.asarray(k, np.float64), np.asarray(v, np.float64)
    alpha, beta = np.asarray(alpha, np.float64), np.asarray(beta, np.float64)
    T, H, dk = q.shape
    dv = v.shape[2]
    o = np.zeros((T, H, dv))
    row = 0
    for i, C in enumerate(int(c) for c in chunk_lens):
        P = 0 if prefix_lens is None else int(prefix_lens[i])
        S = np.zeros((H, dk, dv)) if state_in[i] < 0 else state_pool[state_in[i]].copy()
        n_snap = 0
        for t in range(C):
            r = row + t
            for h in range(H):
                S[h], o[r, h] = kda_step(S[h], q[r, h], k[r, h], v[r, h], alpha[r, h], beta[r, h])
            pos = P + t + 1                               # tokens of the sequence folded into S so far
            if snap_interval > 0 and pos % snap_interval == 0:
                if snap_slots is not None and n_snap < snap_slots.shape[1] and snap_slots[i, n_snap] >= 0:
                    state_pool[snap_slots[i, n_snap]] = S
                n_snap += 1
        if state_out[i] >= 0:
            state_pool[state_out[i]] = S
        row += C
    return o


def snapshot_bytes(bytes_per_element, heads, d_k, d_v, layers=1):
    """Section 3.2's storage of one checkpoint: b * sum over linear layers of H d_k d_v."""
    return bytes_per_element * layers * heads * d_k * d_v
