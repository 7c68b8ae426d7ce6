"""Multi-GPU plumbing for independent replicas.

The synchronisation stage holds all K particles of a swarm on one GPU and has
no exchange step between GPUs, so N GPUs run N independent swarms.  The only
communication is the timing protocol: a barrier on both sides of the timed
region and the maximum of the elapsed time over ranks.  One process per GPU,
``torch.distributed`` (NCCL on GPUs, gloo on CPU for tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class Ranks:
    rank: int = 0
    world: int = 1
    local_rank: int = 0
    backend: str | None = None

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def init_from_env(backend: str | None = None) -> Ranks:
    """Join the process group described by RANK / WORLD_SIZE / MASTER_* if the
    launcher set them; otherwise a single-rank stand-in without a group."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return Ranks()
    rank = int(os.environ["RANK"])
    local = int(os.environ.get("LOCAL_RANK", rank))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend is None:
        # PSOPS_DIST_BACKEND=gloo lets independent replicas rendezvous over CPU
        # tensors, e.g. several replicas sharing one GPU on a development box.
        backend = os.environ.get("PSOPS_DIST_BACKEND") or ("nccl" if torch.cuda.is_available() else "gloo")
    if backend == "nccl":
        torch.cuda.set_device(local)
    dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return Ranks(rank, world, local, backend)


def _device(r: Ranks) -> torch.device:
    return torch.device("cuda", r.local_rank) if r.backend == "nccl" else torch.device("cpu")


def barrier(r: Ranks) -> None:
    if r.world > 1:
        if r.backend == "nccl":
            dist.barrier(device_ids=[r.local_rank])
        else:
            dist.barrier()


def max_over_ranks(r: Ranks, value: float) -> float:
    if r.world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device(r))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(r: Ranks, value: float) -> float:
    if r.world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device(r))
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(r: Ranks, units_this_rank: float, seconds_this_rank: float) -> tuple[float, float]:
    """(units per second of the whole job, slowest rank's seconds): all ranks'
    units divided by the maximum elapsed time."""
    slowest = max_over_ranks(r, seconds_this_rank)
    units = sum_over_ranks(r, units_this_rank)
    return units / slowest, slowest


def finish(r: Ranks) -> None:
    if r.world > 1 and dist.is_initialized():
        dist.destroy_process_group()
