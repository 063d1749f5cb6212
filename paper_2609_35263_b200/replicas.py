"""Multi-GPU plumbing for a path that does not shard: N independent replicas, one process per GPU.

The attention path of one pipeline stage lives on one GPU and has no exchange step, so there is no data-path
collective.  Ranks only meet at a barrier on both sides of the timed region and to take the maximum of their
device-measured times; the whole-job throughput is (units all replicas processed) / (that maximum).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def env_ranks() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: Optional[str] = None, device: Optional[torch.device] = None) -> Tuple[int, int, int]:
    """Join the process group when WORLD_SIZE > 1 (nccl on GPUs, gloo on CPU)."""
    rank, local_rank, world = env_ranks()
    if world > 1 and not torch.distributed.is_initialized():
        backend = backend or ("nccl" if torch.cuda.is_available() else "gloo")
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        torch.distributed.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier(sync_cuda: bool = True) -> None:
    """Device sync, rank barrier, device sync: nothing of the timed region is in flight on either side."""
    if sync_cuda and torch.cuda.is_available():
        torch.cuda.synchronize()
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.barrier()
    if sync_cuda and torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(x: float, device="cpu") -> float:
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_replica: float, ms_per_step_local: float, device="cpu") -> Tuple[float, float]:
    """(whole-job units per second, max-over-ranks ms per step) for replicas doing equal work."""
    world = torch.distributed.get_world_size() if (torch.distributed.is_available() and
                                                   torch.distributed.is_initialized()) else 1
    ms = max_over_ranks(ms_per_step_local, device)
    return world * units_per_replica / (ms * 1e-3), ms


def finalize() -> None:
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.destroy_process_group()
