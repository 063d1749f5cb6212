"""Shared test plumbing: materialise a workload on the CPU and run the oracle on it."""
import numpy as np
import torch

import oracle


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 view of its bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)


def f64(a) -> np.ndarray:
    if isinstance(a, np.ndarray) and a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.detach().cpu().to(torch.float64).numpy()


def cpu_inputs(w):
    return dict(q=w.q(), k_new=w.k_new(), v_new=w.v_new(), k_pool=w.k_pool(), v_pool=w.v_pool())


def run_oracle(w, inp=None, sm_scale=None):
    """Oracle append followed by oracle attention on the appended pools."""
    inp = inp or cpu_inputs(w)
    kp, vp = oracle.oracle_append(inp["k_new"], inp["v_new"], inp["k_pool"], inp["v_pool"],
                                  w.block_tables, w.prefix_lens, w.chunk_lens)
    out, lse = oracle.oracle_attention(inp["q"], kp, vp, w.block_tables, w.prefix_lens, w.chunk_lens,
                                       sm_scale=sm_scale)
    return kp, vp, out, lse
