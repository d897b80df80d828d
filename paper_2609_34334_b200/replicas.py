"""Process plumbing for runs with more than one GPU.

The ring path models its R ranks inside ONE GPU, so it does not shard: with N GPUs the benchmark runs
N independent replicas (one process per GPU) and there is no data-path collective.  torch.distributed
is used only to line the replicas up (barrier) and to combine their timings (max over ranks) and unit
counts (sum over ranks).  Backend "nccl" on GPUs, "gloo" in CPU tests.
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch


@dataclass
class World:
    rank: int = 0
    local_rank: int = 0
    size: int = 1
    backend: str = ""

    @property
    def distributed(self) -> bool:
        return self.size > 1


def init_from_env(backend: str | None = None) -> World:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (as set by torchrun)."""
    size = int(os.environ.get("WORLD_SIZE", "1"))
    if size <= 1:
        return World()
    import torch.distributed as dist

    rank = int(os.environ["RANK"])
    local_rank = int(os.environ.get("LOCAL_RANK", rank))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    if backend == "nccl":
        torch.cuda.set_device(local_rank)
    if not dist.is_initialized():
        kwargs = {}
        if backend == "nccl":
            kwargs["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=size, **kwargs)
    return World(rank, local_rank, size, backend)


def _dev(world: World):
    return torch.device("cuda", world.local_rank) if world.backend == "nccl" else torch.device("cpu")


def barrier(world: World) -> None:
    if world.distributed:
        import torch.distributed as dist

        if world.backend == "nccl":
            dist.barrier(device_ids=[world.local_rank])
        else:
            dist.barrier()


def max_over_ranks(world: World, value: float) -> float:
    if not world.distributed:
        return float(value)
    import torch.distributed as dist

    t = torch.tensor([float(value)], dtype=torch.float64, device=_dev(world))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(world: World, value: float) -> float:
    if not world.distributed:
        return float(value)
    import torch.distributed as dist

    t = torch.tensor([float(value)], dtype=torch.float64, device=_dev(world))
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(world: World, units_this_rank: float, seconds_this_rank: float) -> float:
    """Units all replicas processed divided by the slowest replica's time."""
    total_units = sum_over_ranks(world, units_this_rank)
    slowest = max_over_ranks(world, seconds_this_rank)
    return total_units / slowest if slowest > 0 else 0.0


def shutdown(world: World) -> None:
    if world.distributed:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()
