"""TEST INFRASTRUCTURE — brute-force dense causal attention in numpy fp64 (matrix form).

Written separately from the C oracle, in a different shape (whole-sequence
matrices instead of row streaming), so that it can pin it on tiny inputs:
gather a request's K/V into contiguous arrays, build the full (P+C) x (P+C)
lower-triangular softmax of one-shot causal attention over the whole sequence,
and keep the last C rows.
"""
from __future__ import annotations

import math

import numpy as np


def _to_f64(x) -> np.ndarray:
    """bf16 tensor / uint16 bit patterns -> float64, exactly."""
    if isinstance(x, np.ndarray) and x.dtype == np.uint16:
        return (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    import torch
    if isinstance(x, torch.Tensor):
        return x.to(torch.float64).numpy()
    return np.asarray(x, dtype=np.float64)


def gather_contiguous(pool, block_table_row, n_tokens):
    """pool [num_pages, Hkv, B, d] -> [n_tokens, Hkv, d] following one block-table row."""
    pool = _to_f64(pool)
    _, Hkv, B, d = pool.shape
    nb = (n_tokens + B - 1) // B
    pages = np.asarray(block_table_row[:nb], dtype=np.int64)
    x = pool[pages]                       # [nb, Hkv, B, d]
    x = np.transpose(x, (0, 2, 1, 3)).reshape(nb * B, Hkv, d)
    return x[:n_tokens]


def brute_dense(q, k_pool, v_pool, block_tables, prefix_lens, chunk_lens, sm_scale=None):
    """Returns (out [T, Hq, d], lse [T, Hq]) in float64 via full-sequence dense causal attention.

    Rows of the prefix have no query in this call; their query rows are filled with
    zeros so that the full square problem can be formed, and are dropped afterwards.
    """
    qf = _to_f64(q)
    T, Hq, d = qf.shape
    Hkv = k_pool.shape[1]
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if not sm_scale else float(sm_scale)
    out = np.zeros((T, Hq, d))
    lse = np.zeros((T, Hq))
    off = 0
    for i, (P, C) in enumerate(zip(np.asarray(prefix_lens).tolist(), np.asarray(chunk_lens).tolist())):
        n = P + C
        if C == 0:
            continue
        K = gather_contiguous(k_pool, block_tables[i], n)
        V = gather_contiguous(v_pool, block_tables[i], n)
        tri = np.tril(np.ones((n, n), dtype=bool))
        for h in range(Hq):
            g = h // G
            Qfull = np.zeros((n, d))
            Qfull[P:] = qf[off:off + C, h]
            S = scale * (Qfull @ K[:, g].T)
            S = np.where(tri, S, -np.inf)
            m = S.max(axis=1, keepdims=True)
            W = np.exp(S - m)
            den = W.sum(axis=1, keepdims=True)
            O = (W / den) @ V[:, g]
            out[off:off + C, h] = O[P:]
            lse[off:off + C, h] = (m + np.log(den))[P:, 0]
        off += C
    return out, lse
