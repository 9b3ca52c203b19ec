"""Multi-GPU plumbing: the decoding loop shards by group with no data-path collective, so N GPUs
run N independent replicas (one process per GPU).  The only cross-rank steps are the barrier
around a timed region and the reduction of the per-rank figures: time = max over ranks,
tokens = sum over ranks.  Works with any torch.distributed backend (nccl on GPUs, gloo on CPU)."""
from __future__ import annotations

import json
import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence, Tuple

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


def launch_local(cmd: Sequence[str], n: int, extra_env: Optional[dict] = None, timeout: Optional[float] = None) -> int:
    """Starts `cmd` n times on this node, one process per rank (RANK = LOCAL_RANK = 0..n-1, WORLD_SIZE = n,
    rendezvous on 127.0.0.1 at a free port), waits for all of them and returns the largest exit code.
    The children inherit stdout/stderr, so whatever rank 0 prints is the job's output.  If one rank fails
    the others are terminated (they would wait at the next barrier for ever)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs: List[subprocess.Popen] = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen(list(cmd), env=env))
    rc = 0
    pending = list(procs)
    import time
    t0 = time.time()
    while pending:
        for p in list(pending):
            code = p.poll()
            if code is None:
                continue
            pending.remove(p)
            rc = max(rc, abs(code))
            if code != 0:
                for q in pending:
                    q.terminate()
        if timeout is not None and time.time() - t0 > timeout:
            for q in pending:
                q.terminate()
            rc = max(rc, 124)
            timeout = None
        time.sleep(0.05)
    return rc


def _stub_workload() -> None:
    """Stand-in workload for the launcher's CPU test: every rank joins (gloo), takes its block of 10 groups,
    "times" a step, and rank 0 prints the reduced figures as one JSON line."""
    dist, rank, world = init("gloo")
    groups = list(shard_groups(10, rank, world))
    barrier(dist)
    ms, tokens = reduce_step(dist, 3.0 + rank, 10 * len(groups))
    ranks = reduce_step(dist, 0.0, 1)[1]
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ranks_seen": ranks, "ms": ms, "tokens": tokens, "groups_rank0": groups}))
    barrier(dist)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    if "--stub-workload" in sys.argv:
        if "--fail-rank" in sys.argv and os.environ.get("RANK") == sys.argv[sys.argv.index("--fail-rank") + 1]:
            sys.exit(3)
        _stub_workload()
