"""The step after the hot path, for two ranks: KV-head sharding of the attention calls, and the data-plane hand-off
of a wave (its chunk spans and activations) from one pipeline stage to the next (Section 4.1 "data plane", Section
4.6 chunk spans).  One process per GPU over torch.distributed (nccl on GPUs, gloo on CPU); plumbing only - every
step of the path still runs in the library's kernels.

KV-head sharding needs no exchange inside attention: heads are independent, so rank r runs the same calls on KV
heads [r Hkv/W, (r+1) Hkv/W) and their query heads through strided views of the same tensors.

The hand-off is asynchronous point-to-point: a fixed-size header (wave id, span count, token count, the spans as
(request id, starting token, length)) followed by the activations, received into a ring of buffers so that wave w+1
arrives while wave w computes.  A follower checks every span against the tokens it has itself materialised for that
request and fails the wave on a mismatch (Section 4.6)."""
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
    """Sends waves to the next stage and receives them from the previous one."""

    HEADER = 4           # wave id, number of spans, number of tokens, hidden size

    def __init__(self, rank: int, world: int, hidden: int, max_lanes: int, max_wave_tokens: int,
                 dtype=torch.bfloat16, device="cpu", depth: int = 2):
        self.rank, self.world, self.hidden, self.max_lanes = rank, world, hidden, max_lanes
        self.prev = rank - 1 if rank > 0 else None
        self.next = rank + 1 if rank + 1 < world else None
        self.device = torch.device(device)
        self._hdr = [torch.zeros(self.HEADER + 3 * max_lanes, dtype=torch.int64, device=self.device) for _ in range(depth)]
        self._act = [torch.empty((max_wave_tokens, hidden), dtype=dtype, device=self.device) for _ in range(depth)]
        self._slot = 0
        self._posted = None          # (slot, work) of the header receive in flight
        self._sent: List = []        # (work handles, tensors kept alive)

    # ---- towards the next stage
    def send_wave(self, wave_id: int, spans: Sequence[Span], activations: torch.Tensor) -> None:
        if self.next is None:
            raise RuntimeError("the last stage has nowhere to send")
        n = len(spans)
        if n > self.max_lanes or activations.shape[0] != sum(s[2] for s in spans) or activations.shape[1] != self.hidden:
            raise ValueError("wave does not fit the link or spans and activations disagree")
        hdr = torch.zeros(self.HEADER + 3 * self.max_lanes, dtype=torch.int64)
        hdr[:4] = torch.tensor([wave_id, n, activations.shape[0], self.hidden])
        if n:
            hdr[4:4 + 3 * n] = torch.tensor(spans, dtype=torch.int64).reshape(-1)
        hdr = hdr.to(self.device)
        works = [dist.isend(hdr, self.next)]
        if activations.shape[0]:
            works.append(dist.isend(activations, self.next))
        self._sent.append((works, (hdr, activations)))
        self._sent = [s for s in self._sent if not all(w.is_completed() for w in s[0])]

    def flush(self) -> None:
        for works, _ in self._sent:
            for w in works:
                w.wait()
        self._sent = []

    # ---- from the previous stage
    def post_recv(self) -> None:
        """Start receiving the next wave's header; call it before computing the current wave."""
        if self.prev is None:
            raise RuntimeError("the first stage has nothing to receive")
        if self._posted is None:
            slot = self._slot
            self._posted = (slot, dist.irecv(self._hdr[slot], self.prev))

    def recv_wave(self):
        """(wave id, spans, activations) of the next wave; the activations are a view of a ring buffer that stays
        valid until `depth - 1` further waves have been received."""
        self.post_recv()
        slot, work = self._posted
        work.wait()
        self._posted = None
        self._slot = (slot + 1) % len(self._hdr)
        hdr = self._hdr[slot].cpu()
        wave_id, n, tokens, hidden = (int(x) for x in hdr[:4])
        if hidden != self.hidden or n > self.max_lanes or tokens > self._act[slot].shape[0]:
            raise ValueError("incoming wave does not fit the link")
        spans = [tuple(int(x) for x in hdr[4 + 3 * i:7 + 3 * i]) for i in range(n)]
        act = self._act[slot][:tokens]
        if tokens:
            dist.recv(act, self.prev)
        return wave_id, spans, act
