"""Multi-process plumbing: one process per GPU.

Scheduling rounds of different clusters are independent problems, so in the benchmark ranks
only meet to agree on the timing: a barrier on both sides of the timed region, the MAX over
ranks of the elapsed time and the SUM of the units processed.

One population can also be evolved by several ranks (`evolve_sharded`): the children of a
generation are independent given the parents, so every rank makes and evaluates a contiguous
slice of them and the slices are gathered (the one exchange step of the path: an all-gather
of matrices and fitness) before the next generation.  The result equals the single-process
search bit for bit.  Works with `nccl` (CUDA tensors) and `gloo` (CPU tensors).
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


def all_gather_slices(local, total: int, world: int, rank: int):
    """Concatenation over ranks of per-rank slices of unequal length (rank r holds the rows
    shard_range(total, r, world) of the result).  Single process: returns `local`."""
    import torch
    import torch.distributed as dist

    if world == 1 or not (dist.is_available() and dist.is_initialized()):
        return local
    longest = shard_range(total, 0, world)
    longest = longest[1] - longest[0]
    padded = torch.zeros((longest,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    padded[: local.shape[0]] = local
    raw = padded.view(torch.uint8)                 # bytes: every backend gathers them, whatever the element type
    parts = [torch.empty_like(raw) for _ in range(world)]
    dist.all_gather(parts, raw)
    out = []
    for r in range(world):
        b, e = shard_range(total, r, world)
        out.append(parts[r].view(local.dtype).view(padded.shape)[: e - b])
    return torch.cat(out)


def evolve_sharded(make_children, evaluate, pop, fit, generations: int, rank: int, world: int, first_generation: int = 0):
    """`generations` generations of one population over `world` ranks.

    make_children(pop, fit, first_child, num_children, generation) -> the children's matrices,
    evaluate(children) -> their fitness (both for this rank's slice only; on a GPU these are
    Scheduler.ga_generation_shard and Scheduler.eval_fitness).  pop / fit: all parents, identical
    on every rank.  Returns the final (pop, fit), again identical on every rank."""
    P = pop.shape[0]
    b, e = shard_range(P, rank, world)
    for g in range(first_generation, first_generation + generations):
        children = make_children(pop, fit, b, e - b, g)
        cfit = evaluate(children)
        pop = all_gather_slices(children, P, world, rank)
        fit = all_gather_slices(cfit, P, world, rank)
    return pop, fit
