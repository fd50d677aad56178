"""Multi-process plumbing for the benchmark: one process per GPU, no data-path collective.

Scheduling rounds of different clusters (and candidates of one population) are independent
problems, so ranks only meet to agree on the timing: a barrier on both sides of the timed
region, the MAX over ranks of the elapsed time and the SUM of the units processed.  Works
with `nccl` (CUDA tensors) and `gloo` (CPU tensors).
"""
from __future__ import annotations

import os


def env_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str):
    """Initialise torch.distributed from the torchrun environment when WORLD_SIZE > 1."""
    import torch.distributed as dist

    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def shard_range(total: int, rank: int, world: int):
    """Contiguous, balanced [begin, end) slice of `total` independent units for `rank`."""
    base, rem = divmod(total, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def aggregate(elapsed_ms: float, units: float, device="cpu"):
    """(max over ranks of elapsed_ms, sum over ranks of units)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(elapsed_ms: float, units: float, device="cpu"):
    """Whole-job throughput in units per second: all ranks' units over the slowest rank's time."""
    t, u = aggregate(elapsed_ms, units, device)
    return (u / (t * 1e-3)) if t > 0 else 0.0, t, u
