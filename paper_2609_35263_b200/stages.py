"""The step after the hot path, for two ranks: KV-head sharding of the attention calls, and the data-plane hand-off
of a wave (its chunk spans and activations) from one pipeline stage to the next (Section 4.1 "data plane", Section
4.6 chunk spans).  One process per GPU over torch.distributed (nccl on GPUs, gloo on CPU); plumbing only - every
step of the path still runs in the library's kernels.

KV-head sharding needs no exchange inside attention: heads are independent, so rank r runs the same calls on KV
heads [r Hkv/W, (r+1) Hkv/W) and their query heads through strided views of the same tensors.

The hand-off is asynchronous point-to-point: a fixed-size header (wave id, span count, token count, the spans as
(request id, starting token, length)) and the activations.  Both messages have a fixed size (the activations always
travel as the link's full wave buffer, `max_wave_tokens` rows, of which the header says how many count), so a stage
can post both receives of wave w+1 before it knows anything about that wave, i.e. before it starts computing wave
w: the transfer overlaps the compute.  Waves are planned to fill the budget, so little of the buffer is padding.  A
follower checks every span against the tokens it has itself materialised for that request and fails the wave on a
mismatch (Section 4.6)."""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import torch
import torch.distributed as dist

from .binding import WppError, make_desc

WPP_ERR_POSITION_MISMATCH = 4
Span = Tuple[int, int, int]          # (request id, starting token, length)


def head_shard(rank: int, world: int, num_requests: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
               page_size: int, max_blocks_per_req: int, num_pages: int, q, out, k_new, v_new, k_pool, v_pool):
    """(desc, views) for rank `rank` of `world` KV-head shards: strided views of q/out [T, Hq, d], k_new/v_new
    [T, Hkv, d] and the pools [pages, Hkv, B, d]; the descriptor carries the parents' strides."""
    if num_kv_heads % world or not 0 <= rank < world:
        raise ValueError("KV heads must divide evenly over the shards")
    hk = num_kv_heads // world
    hq = hk * (num_q_heads // num_kv_heads)
    ks, qs = slice(rank * hk, (rank + 1) * hk), slice(rank * hq, (rank + 1) * hq)
    desc = make_desc(num_requests, hq, hk, head_dim, page_size, max_blocks_per_req, num_pages,
                     kv_page_stride=k_pool.stride(0), kv_head_stride=k_pool.stride(1), kv_token_stride=k_pool.stride(2),
                     q_token_stride=q.stride(0), q_head_stride=q.stride(1),
                     kvnew_token_stride=k_new.stride(0), kvnew_head_stride=k_new.stride(1),
                     o_token_stride=out.stride(0), o_head_stride=out.stride(1))
    views = dict(q=q[:, qs], out=out[:, qs], k_new=k_new[:, ks], v_new=v_new[:, ks], k_pool=k_pool[:, ks],
                 v_pool=v_pool[:, ks])
    return desc, views


def check_spans(spans: Sequence[Span], materialised: Dict[int, int]) -> None:
    """Section 4.6: a span must start exactly where this rank's own cache of the request ends; otherwise the wave
    fails.  On success the positions advance by the spans' lengths."""
    for req, start, length in spans:
        if length < 0 or materialised.get(req, 0) != start:
            raise WppError(WPP_ERR_POSITION_MISMATCH,
                           f"span of request {req} starts at {start}, {materialised.get(req, 0)} tokens are cached")
    for req, start, length in spans:
        materialised[req] = start + length


class StageLink:
    """Sends waves to the next stage and receives them from the previous one (a middle stage does both)."""

    HEADER = 4           # wave id, number of spans, number of tokens, hidden size

    def __init__(self, rank: int, world: int, hidden: int, max_lanes: int, max_wave_tokens: int,
                 dtype=torch.bfloat16, device="cpu", depth: int = 2):
        self.rank, self.world, self.hidden, self.max_lanes = rank, world, hidden, max_lanes
        self.prev = rank - 1 if rank > 0 else None
        self.next = rank + 1 if rank + 1 < world else None
        self.device = torch.device(device)
        hdr = lambda: torch.zeros(self.HEADER + 3 * max_lanes, dtype=torch.int64, device=self.device)
        act = lambda: torch.zeros((max_wave_tokens, hidden), dtype=dtype, device=self.device)
        self._hdr = [hdr() for _ in range(depth)] if self.prev is not None else []
        self._act = [act() for _ in range(depth)] if self.prev is not None else []
        self._slot = 0
        self._posted = None          # (slot, header work, activation work) of the receives in flight
        # send side: a ring of staging buffers; a buffer is reused once its two sends have completed
        self._out_hdr = [hdr() for _ in range(depth)] if self.next is not None else []
        self._out_act = [act() for _ in range(depth)] if self.next is not None else []
        self._out_work: List = [None] * depth
        self._out_slot = 0

    # ---- towards the next stage
    def send_wave(self, wave_id: int, spans: Sequence[Span], activations: torch.Tensor) -> None:
        if self.next is None:
            raise RuntimeError("the last stage has nowhere to send")
        n = len(spans)
        tokens = int(activations.shape[0])
        if (n > self.max_lanes or tokens != sum(s[2] for s in spans) or activations.shape[1] != self.hidden
                or tokens > self._out_act[0].shape[0]):
            raise ValueError("wave does not fit the link or spans and activations disagree")
        slot = self._out_slot
        self._out_slot = (slot + 1) % len(self._out_hdr)
        if self._out_work[slot] is not None:
            for w in self._out_work[slot]:
                w.wait()
        hdr = torch.zeros(self.HEADER + 3 * self.max_lanes, dtype=torch.int64)
        hdr[:4] = torch.tensor([wave_id, n, tokens, self.hidden])
        if n:
            hdr[4:4 + 3 * n] = torch.tensor(spans, dtype=torch.int64).reshape(-1)
        self._out_hdr[slot].copy_(hdr)
        self._out_act[slot][:tokens].copy_(activations)
        self._out_work[slot] = [dist.isend(self._out_hdr[slot], self.next), dist.isend(self._out_act[slot], self.next)]

    def flush(self) -> None:
        for i, works in enumerate(self._out_work):
            if works is not None:
                for w in works:
                    w.wait()
                self._out_work[i] = None

    # ---- from the previous stage
    def post_recv(self) -> None:
        """Start receiving the next wave, header and activations; call it before computing the current wave so
        that the transfer runs under the compute."""
        if self.prev is None:
            raise RuntimeError("the first stage has nothing to receive")
        if self._posted is None:
            slot = self._slot
            self._posted = (slot, dist.irecv(self._hdr[slot], self.prev), dist.irecv(self._act[slot], self.prev))

    def recv_wave(self):
        """(wave id, spans, activations) of the next wave; the activations are a view of a ring buffer that stays
        valid until `depth - 1` further receives have been posted."""
        self.post_recv()
        slot, hdr_work, act_work = self._posted
        hdr_work.wait()
        act_work.wait()
        self._posted = None
        self._slot = (slot + 1) % len(self._hdr)
        hdr = self._hdr[slot].cpu()
        wave_id, n, tokens, hidden = (int(x) for x in hdr[:4])
        if hidden != self.hidden or n > self.max_lanes or tokens > self._act[slot].shape[0]:
            raise ValueError("incoming wave does not fit the link")
        spans = [tuple(int(x) for x in hdr[4 + 3 * i:7 + 3 * i]) for i in range(n)]
        return wave_id, spans, self._act[slot][:tokens]
