"""Seeded workload descriptions and counter-based bf16 value streams.

Lengths and page ids come from ``numpy.random.default_rng(seed)`` in a fixed
draw order.  Values come from a counter-based generator (an integer hash of
(seed, stream, linear index) looked up in a 65536-entry table of normal
quantiles), so that any slice of any tensor can be produced on the CPU or on
a CUDA device with identical bits and without materialising the rest.

Pools are filled *by physical address*: element (page, kv_head, slot, e) of
the K pool is a pure function of its linear index in the pool.  A request's
cached prefix is therefore simply whatever its block table points at, pages
shared by several block tables are shared for real, and no page gather or
scatter happens in this module.
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Dict, Optional

import numpy as np
import torch

STREAM_Q, STREAM_KNEW, STREAM_VNEW, STREAM_KPOOL, STREAM_VPOOL = 0, 1, 2, 3, 4

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _signed(x: int) -> int:
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _py_mix(x: int) -> int:
    x &= _M64
    x = ((x ^ (x >> 30)) * _C1) & _M64
    x = ((x ^ (x >> 27)) * _C2) & _M64
    return x ^ (x >> 31)


_TABLE_CPU: Optional[torch.Tensor] = None
_TABLE_DEV: Dict[str, torch.Tensor] = {}


def _normal_table(device) -> torch.Tensor:
    """65536 mid-point quantiles of N(0,1), rounded to bf16 (always computed on the CPU)."""
    global _TABLE_CPU
    if _TABLE_CPU is None:
        u = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _TABLE_CPU = torch.special.ndtri(u).to(torch.bfloat16)
    key = str(device)
    if key not in _TABLE_DEV:
        _TABLE_DEV[key] = _TABLE_CPU.to(device)
    return _TABLE_DEV[key]


def counter_normal_bf16(seed: int, stream: int, start: int, count: int, device="cpu",
                        block: int = 1 << 25) -> torch.Tensor:
    """bf16 values for linear indices [start, start+count) of stream ``stream``."""
    device = torch.device(device)
    table = _normal_table(device)
    key = _signed(_py_mix((seed * _GOLDEN + stream * 0xD1B54A32D192ED03 + 0x1234567) & _M64))
    out = torch.empty(count, dtype=torch.bfloat16, device=device)
    g, c1, c2 = _signed(_GOLDEN), _signed(_C1), _signed(_C2)
    for s in range(0, count, block):
        n = min(block, count - s)
        x = torch.arange(start + s, start + s + n, dtype=torch.int64, device=device)
        x = x * g + key
        x = (x ^ ((x >> 30) & ((1 << 34) - 1))) * c1
        x = (x ^ ((x >> 27) & ((1 << 37) - 1))) * c2
        x = x ^ ((x >> 31) & ((1 << 33) - 1))
        idx = (x >> 48) & 0xFFFF
        out[s:s + n] = table[idx]
    return out


@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    prefix_lens: np.ndarray          # int32 [R]
    chunk_lens: np.ndarray           # int32 [R]
    block_tables: np.ndarray         # int32 [R, max_blocks]; unused entries are -1
    num_pages: int
    page_scale_log2: Optional[np.ndarray] = None    # int32 [num_pages]: K rows of the page are scaled by 2**this
    token_scale_log2: Optional[np.ndarray] = None   # int32 [T]: new K rows are scaled by 2**this
    notes: str = ""

    # ---- shapes -------------------------------------------------------
    @property
    def num_requests(self) -> int:
        return int(self.prefix_lens.shape[0])

    @property
    def max_blocks_per_req(self) -> int:
        return int(self.block_tables.shape[1])

    @property
    def total_new_tokens(self) -> int:
        return int(self.chunk_lens.astype(np.int64).sum())

    @property
    def q_offsets(self) -> np.ndarray:
        off = np.zeros(self.num_requests + 1, dtype=np.int64)
        np.cumsum(self.chunk_lens.astype(np.int64), out=off[1:])
        return off

    @property
    def visible_pairs(self) -> int:
        """Visible (query, key) pairs per query head: sum C*P + C(C+1)/2."""
        P = self.prefix_lens.astype(np.int64)
        C = self.chunk_lens.astype(np.int64)
        return int((C * P + C * (C + 1) // 2).sum())

    @property
    def flops(self) -> int:
        return 4 * self.head_dim * self.num_q_heads * self.visible_pairs

    def unique_kv_pages(self) -> int:
        used = self.block_tables[self.block_tables >= 0]
        return int(np.unique(used).size)

    # ---- values -------------------------------------------------------
    def _stream(self, stream, shape, device, start_row=0, rows=None):
        inner = int(np.prod(shape[1:]))
        n_rows = shape[0] if rows is None else rows
        flat = counter_normal_bf16(self.seed, stream, start_row * inner, n_rows * inner, device)
        return flat.view(n_rows, *shape[1:])

    def q(self, device="cpu", start_row=0, rows=None) -> torch.Tensor:
        """[T, Hq, d] bf16 (or rows [start_row, start_row+rows) of it)."""
        return self._stream(STREAM_Q, (self.total_new_tokens, self.num_q_heads, self.head_dim),
                            device, start_row, rows)

    def _scaled(self, t: torch.Tensor, log2: Optional[np.ndarray], start_row: int) -> torch.Tensor:
        if log2 is None:
            return t
        e = torch.from_numpy(log2[start_row:start_row + t.shape[0]].astype(np.float32)).to(t.device)
        f = torch.exp2(e).to(torch.bfloat16)       # a power of two: exact in bf16
        return t * f.view(-1, *([1] * (t.dim() - 1)))

    def k_new(self, device="cpu", start_row=0, rows=None) -> torch.Tensor:
        """[T, Hkv, d] bf16: the chunk's keys, in request order."""
        t = self._stream(STREAM_KNEW, (self.total_new_tokens, self.num_kv_heads, self.head_dim),
                         device, start_row, rows)
        return self._scaled(t, self.token_scale_log2, start_row)

    def v_new(self, device="cpu", start_row=0, rows=None) -> torch.Tensor:
        return self._stream(STREAM_VNEW, (self.total_new_tokens, self.num_kv_heads, self.head_dim),
                            device, start_row, rows)

    def k_pool(self, device="cpu", start_page=0, pages=None) -> torch.Tensor:
        """[num_pages, Hkv, B, d] bf16, filled by physical address (cached prefix + stale slots)."""
        t = self._stream(STREAM_KPOOL, (self.num_pages, self.num_kv_heads, self.page_size, self.head_dim),
                         device, start_page, pages)
        return self._scaled(t, self.page_scale_log2, start_page)

    def v_pool(self, device="cpu", start_page=0, pages=None) -> torch.Tensor:
        return self._stream(STREAM_VPOOL, (self.num_pages, self.num_kv_heads, self.page_size, self.head_dim),
                            device, start_page, pages)

    def summary(self) -> dict:
        return {
            "name": self.name, "seed": self.seed, "requests": self.num_requests,
            "new_tokens": self.total_new_tokens,
            "served_tokens": int((self.prefix_lens.astype(np.int64) + self.chunk_lens).sum()),
            "q_heads": self.num_q_heads, "kv_heads": self.num_kv_heads, "head_dim": self.head_dim,
            "page_size": self.page_size, "num_pages": self.num_pages,
            "unique_kv_pages": self.unique_kv_pages(), "visible_pairs_per_head": self.visible_pairs,
            "flops": self.flops,
        }


def _blocks(n, B):
    return (np.asarray(n, dtype=np.int64) + B - 1) // B


def make_workload(name, seed, rng, prefix_lens, chunk_lens, Hq, Hkv, d, B,
                  shared_tokens=0, sharers=None, k_scale: Optional[str] = None,
                  spare_pages=64, notes="") -> Workload:
    """Assign physical pages (shared pages first, then request by request) from one permutation."""
    P = np.asarray(prefix_lens, dtype=np.int64)
    C = np.asarray(chunk_lens, dtype=np.int64)
    R = P.shape[0]
    sharers = np.zeros(R, dtype=bool) if sharers is None else np.asarray(sharers, dtype=bool)
    assert shared_tokens % B == 0, "a shared page must be a full page"
    assert np.all(P[sharers] >= shared_tokens)
    n_shared = shared_tokens // B if sharers.any() else 0
    blocks = _blocks(P + C, B)
    private = blocks - n_shared * sharers
    needed = int(n_shared + private.sum())
    num_pages = needed + spare_pages
    perm = rng.permutation(num_pages).astype(np.int32)
    max_blocks = int(max(1, blocks.max() if R else 1))
    bt = np.full((R, max_blocks), -1, dtype=np.int32)
    cur = 0
    shared_ids = perm[cur:cur + n_shared]
    cur += n_shared
    for i in range(R):
        nb = int(blocks[i])
        if sharers[i]:
            bt[i, :n_shared] = shared_ids
            bt[i, n_shared:nb] = perm[cur:cur + nb - n_shared]
            cur += nb - n_shared
        else:
            bt[i, :nb] = perm[cur:cur + nb]
            cur += nb
    assert cur == needed
    page_scale = token_scale = None
    if k_scale is not None:
        assert not sharers.any() and 4096 % B == 0
        def expo(pos):
            blk = pos // 4096
            return blk if k_scale == "cumulative" else (blk % 2)
        page_scale = np.zeros(num_pages, dtype=np.int32)
        for i in range(R):
            nb = int(blocks[i])
            page_scale[bt[i, :nb]] = expo(np.arange(nb, dtype=np.int64) * B)
        token_scale = np.concatenate([expo(P[i] + np.arange(C[i], dtype=np.int64)) for i in range(R)]
                                     or [np.zeros(0, dtype=np.int64)]).astype(np.int32)
    return Workload(name=name, seed=seed, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=d, page_size=B,
                    prefix_lens=P.astype(np.int32), chunk_lens=C.astype(np.int32), block_tables=bt,
                    num_pages=num_pages, page_scale_log2=page_scale, token_scale_log2=token_scale,
                    notes=notes)


def custom_workload(prefix_lens, chunk_lens, Hq, Hkv, d, B, seed=0, spare_pages=3, **kw) -> Workload:
    """Small hand-specified cases for tests."""
    rng = np.random.default_rng(seed)
    return make_workload(kw.pop("name", "custom"), seed, rng, prefix_lens, chunk_lens, Hq, Hkv, d, B,
                         spare_pages=spare_pages, **kw)


def cfg1() -> Workload:
    """One request: 256 cached tokens in 16-token pages, 128 new tokens, 8/2 heads, d=64."""
    rng = np.random.default_rng(1)
    return make_workload("cfg1", 1, rng, [256], [128], 8, 2, 64, 16)


def cfg2() -> Workload:
    """16 ragged requests, private page-rounded prefixes up to 8192, chunks 256..2048, 32/8 heads."""
    rng = np.random.default_rng(2)
    pages = rng.integers(0, 129, size=16)
    C = rng.integers(256, 2049, size=16)
    return make_workload("cfg2", 2, rng, pages * 64, C, 32, 8, 128, 64)


def cfg3(num_requests: int = 128) -> Workload:
    """Concurrency 128, high reuse: 80 % of requests share one 16384-token prefix (same physical pages)."""
    rng = np.random.default_rng(3)
    R = num_requests
    perm = rng.permutation(R)
    sharers = np.zeros(R, dtype=bool)
    sharers[perm[: (R * 4) // 5]] = True
    suffix = rng.integers(0, 4097, size=R)
    priv = rng.integers(0, 8193, size=R)
    C = rng.integers(256, 4097, size=R)
    P = np.where(sharers, 16384 + suffix, priv)
    return make_workload("cfg3" if R == 128 else f"cfg3_r{R}", 3, rng, P, C, 64, 8, 128, 64,
                         shared_tokens=16384, sharers=sharers,
                         notes="80% (102 of 128) share a 16384-token prefix; private suffix not page-rounded")


def cfg4(k_scale: str = "cumulative", num_requests: int = 8, prefix: int = 98304, chunk: int = 8192) -> Workload:
    """Long context: K rows scaled by a power of two that changes every 4096 positions."""
    rng = np.random.default_rng(4)
    name = "cfg4" if k_scale == "cumulative" else "cfg4_alt"
    return make_workload(name, 4, rng, [prefix] * num_requests, [chunk] * num_requests, 64, 8, 128, 64,
                         k_scale=k_scale,
                         notes="K scale 2**floor(pos/4096)" if k_scale == "cumulative"
                         else "K scale 2**(floor(pos/4096) mod 2)")


def cfg5_cell(chunk: int, prefix: int, num_requests: int = 32) -> Workload:
    """One cell of the sweep grid: uniform requests, private pages."""
    rng = np.random.default_rng(5)
    return make_workload(f"cfg5_C{chunk}_P{prefix}", 5, rng, [prefix] * num_requests,
                         [chunk] * num_requests, 64, 8, 128, 64)


CONFIG_BUILDERS: Dict[str, Callable[[], Workload]] = {
    "cfg1": cfg1,
    "cfg2": cfg2,
    "cfg3": cfg3,
    "cfg4": cfg4,
    "cfg4_alt": lambda: cfg4("alternate"),
}


# ---------------------------------------------------------------------------------------------------------------
# Inputs of the recurrent-state (KDA) layer.  Only value streams and their pre-processing live here: keys are
# L2-normalised and queries scaled by d_k^-1/2 *before* the operation, as a model does ahead of the update the
# paper prints; decays are sigmoid(4 + 2 n) (median 0.98, a few per cent of channels below 0.9) and write
# strengths sigmoid(n), n standard normal.
STREAM_KDA_Q, STREAM_KDA_K, STREAM_KDA_V, STREAM_KDA_ALPHA, STREAM_KDA_BETA, STREAM_KDA_STATE = 8, 9, 10, 11, 12, 13


@dataclasses.dataclass
class KdaWorkload:
    name: str
    seed: int
    chunk_lens: np.ndarray        # int64 [R]
    prefix_lens: np.ndarray       # int32 [R]: tokens already folded into the resumed state
    num_heads: int
    d_k: int
    d_v: int
    num_slots: int
    state_in: np.ndarray          # int32 [R]
    state_out: np.ndarray         # int32 [R]
    snap_interval: int = 0
    snap_slots: Optional[np.ndarray] = None      # int32 [R, max_snaps]

    @property
    def total_tokens(self) -> int:
        return int(self.chunk_lens.sum())

    @property
    def row_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.chunk_lens)]).astype(np.int64)

    def tensors(self, device="cpu") -> Dict[str, torch.Tensor]:
        """q, k, v (bf16), alpha, beta (fp32) and the state pool (fp32); always computed on the CPU so that the
        bits do not depend on the device, then moved."""
        T, H, dk, dv = self.total_tokens, self.num_heads, self.d_k, self.d_v
        n = lambda stream, count: counter_normal_bf16(self.seed, stream, 0, count).float()
        q = (n(STREAM_KDA_Q, T * H * dk).view(T, H, dk) * dk ** -0.5).to(torch.bfloat16)
        k = n(STREAM_KDA_K, T * H * dk).view(T, H, dk)
        k = (k / k.norm(dim=-1, keepdim=True).clamp_min(1e-6)).to(torch.bfloat16)
        v = n(STREAM_KDA_V, T * H * dv).view(T, H, dv).to(torch.bfloat16)
        alpha = torch.sigmoid(4.0 + 2.0 * n(STREAM_KDA_ALPHA, T * H * dk)).view(T, H, dk).contiguous()
        beta = torch.sigmoid(n(STREAM_KDA_BETA, T * H)).view(T, H).contiguous()
        state = (0.1 * n(STREAM_KDA_STATE, self.num_slots * H * dk * dv)).view(self.num_slots, H, dk, dv).contiguous()
        out = dict(q=q, k=k, v=v, alpha=alpha, beta=beta, state_pool=state)
        return {name: t.to(device) for name, t in out.items()}


def kda_workload(name, seed, chunk_lens, num_heads, prefix_lens=None, resume=None, snap_interval=0, d_k=128,
                 d_v=128, spare_slots=2) -> KdaWorkload:
    """Request i resumes from slot i when resume[i] (default: when its prefix is not empty) and stores its final
    state in slot R + i; periodic snapshots, if any, go to slots after those, one per boundary inside the chunk."""
    chunk_lens = np.asarray(chunk_lens, dtype=np.int64)
    R = int(chunk_lens.size)
    prefix_lens = np.zeros(R, np.int32) if prefix_lens is None else np.asarray(prefix_lens, dtype=np.int32)
    resume = (prefix_lens > 0) if resume is None else np.asarray(resume, dtype=bool)
    state_in = np.where(resume, np.arange(R), -1).astype(np.int32)
    state_out = (R + np.arange(R)).astype(np.int32)
    slots, snaps = 2 * R, None
    if snap_interval > 0:
        counts = (prefix_lens + chunk_lens) // snap_interval - prefix_lens // snap_interval
        snaps = np.full((R, max(1, int(counts.max()) if R else 1)), -1, dtype=np.int32)
        for i in range(R):
            for j in range(int(counts[i])):
                snaps[i, j] = slots
                slots += 1
    return KdaWorkload(name, seed, chunk_lens, prefix_lens, num_heads, d_k, d_v, slots + spare_slots, state_in,
                       state_out, snap_interval, snaps)


def kda_wave(num_requests: int = 8, chunk: int = 2048, num_heads: int = 32, prefix: int = 65536, seed: int = 7) -> KdaWorkload:
    """One wave of a hybrid model's recurrent layer at the paper's matched settings: a 16,384-token budget shared
    by 8 lanes, 32 state heads of 128 x 128, every request resuming from the snapshot of a reused prefix."""
    return kda_workload(f"kda_wave_{num_requests}x{chunk}", seed, [chunk] * num_requests, num_heads,
                        [prefix] * num_requests)
