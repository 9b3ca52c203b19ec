"""Multi-GPU plumbing: the decoding loop shards by group with no data-path collective, so N GPUs
run N independent replicas (one process per GPU).  The only cross-rank steps are the barrier
around a timed region and the reduction of the per-rank figures: time = max over ranks,
tokens = sum over ranks.  Works with any torch.distributed backend (nccl on GPUs, gloo on CPU)."""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def init(backend: Optional[str] = None, device: Optional[torch.device] = None):
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT.
    Returns (dist module or None when WORLD_SIZE == 1, rank, world size)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world == 1:
        return None, 0, 1
    import torch.distributed as dist
    if not dist.is_initialized():
        kwargs = {}
        if device is not None and device.type == "cuda":
            kwargs["device_id"] = device
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"), **kwargs)
    return dist, rank, world


def barrier(dist, device: Optional[torch.device] = None) -> None:
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
        if device is not None and device.type == "cuda":
            torch.cuda.synchronize(device)


def shard_groups(n_groups: int, rank: int, world: int) -> range:
    """Contiguous block of group ids served by this rank (sizes differ by at most one)."""
    base, extra = divmod(n_groups, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def reduce_step(dist, ms: float, tokens: int, device: Optional[torch.device] = None) -> Tuple[float, int]:
    """Whole-job figures of one timed region: (max time over ranks in ms, tokens summed over ranks)."""
    if dist is None:
        return ms, tokens
    dev = device if device is not None else torch.device("cpu")
    t = torch.tensor([ms], dtype=torch.float64, device=dev)
    n = torch.tensor([tokens], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), int(n[0])
