"""Particle-sharded PSO-PS synchronisation across GPUs (one process per GPU).

The paper's Algorithm 3 gathers every worker's full weight vector and loss.
On NVLink/NVSwitch that is unnecessary: all ranks can agree on the best
particle from the K losses alone, so the exchange per sync is one all-gather of
K floats and one broadcast of the best particle's N weights, which lands in
each GPU's own memory before the update kernel reads it (no remote loads in any
kernel).  Bytes received per rank per sync: 4 N + 4 K instead of 4 N (K - 1).

This module only orders collectives and library calls; all arithmetic is in
the CUDA library (``psops_shard_select`` / ``psops_shard_update``).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def owner_of(g: int, counts: list[int]) -> tuple[int, int]:
    """(rank that holds swarm-wide particle g, its row index on that rank) for
    shards holding counts[r] consecutive particles each."""
    first = 0
    for rank, n in enumerate(counts):
        if g < first + n:
            return rank, g - first
        first += n
    raise ValueError(f"particle {g} outside a swarm of {first}")


def first_index(rank: int, counts: list[int]) -> int:
    return sum(counts[:rank])


def bytes_received_per_sync(N: int, counts: list[int]) -> dict:
    """Per-rank traffic of one sync: this exchange vs gathering every particle."""
    K = sum(counts)
    return {"losses_all_gather": 4 * K, "gbest_broadcast": 4 * N,
            "gather_all_particles": 4 * N * (K - max(counts))}


class ShardedSync:
    """Drives one shard.  ``engine`` offers set_losses(all K losses),
    shard_select() -> g, copy_row(local_row, out) and shard_update(gbest, t, lam);
    on GPUs that is a :class:`paper_2009_03816_b200.binding.Swarm` wrapped by
    :func:`swarm_engine`."""

    def __init__(self, engine, counts: list[int], N: int, device, group=None):
        self.engine, self.counts, self.N = engine, list(counts), int(N)
        self.group = group
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        assert len(self.counts) == self.world
        self.K = sum(self.counts)
        self.device = device
        self.gbest = torch.zeros(self.N, dtype=torch.float32, device=device)
        self.all_losses = torch.zeros(self.K, dtype=torch.float32, device=device)

    def sync(self, local_losses: torch.Tensor, t_iter: int = 0, lam: float = 1.0) -> int:
        """local_losses: this rank's counts[rank] losses (tensor on self.device)."""
        if self.world > 1:
            # equal-sized pieces (collectives want them): pad to the largest shard
            widest = max(self.counts)
            mine = torch.zeros(widest, dtype=torch.float32, device=self.device)
            mine[:self.counts[self.rank]] = local_losses.to(self.device, torch.float32)
            pieces = [torch.empty_like(mine) for _ in range(self.world)]
            dist.all_gather(pieces, mine, group=self.group)
            at = 0
            for piece, n in zip(pieces, self.counts):
                self.all_losses[at:at + n] = piece[:n]
                at += n
        else:
            self.all_losses.copy_(local_losses)
        self.engine.set_losses(self.all_losses)
        g = self.engine.shard_select()              # the same on every rank
        owner, row = owner_of(g, self.counts)
        if owner == self.rank:
            self.engine.copy_row(row, self.gbest)
        if self.world > 1:
            dist.broadcast(self.gbest, src=dist.get_global_rank(self.group, owner) if self.group else owner,
                           group=self.group)
        self.engine.shard_update(self.gbest, t_iter, lam)
        return g


def swarm_engine(swarm):
    """Adapter from a binding.Swarm created with k_first / K_total."""
    from . import binding

    class _Engine:
        def set_losses(self, all_losses):
            swarm.set_losses(all_losses)

        def shard_select(self):
            return swarm.shard_select()

        def copy_row(self, row, out):
            binding.psops_get_weights(swarm.ctx, binding.PSOPS_X, row, out)

        def shard_update(self, gbest, t_iter, lam):
            swarm.shard_update(gbest, t_iter, lam)

    return _Engine()
