"""One process per GPU: rendezvous from the torchrun environment and the two reductions the
benchmark needs (max of a time, sum of a count).  With WORLD_SIZE unset everything is a no-op.

Ranks own independent worker groups (their own shard of samples, their own W workers); nothing
on the data path crosses ranks, so no collective runs inside the timed kernels.
"""
from __future__ import annotations

import os

import torch

_initialised = False


def init_from_env(backend: str = "nccl"):
    """Returns (rank, world_size, local_rank); initialises torch.distributed when world_size > 1."""
    global _initialised
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not _initialised:
        import torch.distributed as td
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local)
        td.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
        _initialised = True
    return rank, world, local


def _device():
    import torch.distributed as td
    return torch.device("cuda", torch.cuda.current_device()) if td.get_backend() == "nccl" else torch.device("cpu")


def barrier():
    if _initialised:
        import torch.distributed as td
        td.barrier()


def max_over_ranks(x: float) -> float:
    if not _initialised:
        return float(x)
    import torch.distributed as td
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    td.all_reduce(t, op=td.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    if not _initialised:
        return float(x)
    import torch.distributed as td
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    td.all_reduce(t, op=td.ReduceOp.SUM)
    return float(t.item())


def shard_seed(seed: int, rank: int, world: int) -> int:
    """Seed of a rank's own sample shard (rank 0 of a single-rank job keeps the workload's seed)."""
    return seed + 1000 * rank if world > 1 else seed


def shutdown():
    global _initialised
    if _initialised:
        import torch.distributed as td
        td.destroy_process_group()
        _initialised = False
