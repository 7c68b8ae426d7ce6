"""Particle-sharded PSO-PS synchronisation across GPUs (one process per GPU).

The paper's Algorithm 3 gathers every worker's full weight vector and loss.
On NVLink/NVSwitch that is unnecessary: all ranks can agree on the best
particle from the K losses alone, so the exchange per sync is one all-gather of
K floats and one broadcast of the best particle's N weights, which lands in
each GPU's own memory before the update kernel reads it (no remote loads in any
kernel).  Bytes received per rank per sync: 4 N + 4 K instead of 4 N (K - 1).

The broadcast travels in a few element ranges; the update of a range is
enqueued as soon as that range has arrived, so the transfer of the next range
overlaps it.  The rank that holds the best particle sends the row straight out
of its own weights and also reads gBest from there (every element of gBest is
read by the thread that later overwrites it), so it copies nothing.

This module only orders collectives and library calls; all arithmetic is in
the CUDA library (``psops_shard_select`` / ``psops_shard_update_range``).
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


def range_bounds(N: int, pieces: int, quantum: int = 1024) -> list[tuple[int, int]]:
    """[first, last) element ranges that cover [0, N) left to right: `pieces`
    of them (fewer for a short vector), every boundary but N a multiple of
    `quantum` elements (the library wants multiples of 4; whole KiB keep the
    pieces of a transfer aligned)."""
    pieces = max(1, int(pieces))
    step = -(-N // pieces)                          # ceil
    step = -(-step // quantum) * quantum
    bounds, at = [], 0
    while at < N:
        bounds.append((at, min(N, at + step)))
        at += step
    return bounds


class ShardedSync:
    """Drives one shard.  ``engine`` offers set_losses(all K losses),
    shard_select() -> g, row(local_row) -> the N weights of that row as a tensor
    view, and shard_update_range(gbest, first, last, t, lam); on GPUs that is a
    :class:`paper_2009_03816_b200.binding.Swarm` wrapped by :func:`swarm_engine`.

    ``pieces``: element ranges the gBest broadcast is split into (1 = one
    broadcast, then one update).  ``timing``: record CUDA events around the
    exchange and the update of every sync (see :meth:`timings_ms`)."""

    def __init__(self, engine, counts: list[int], N: int, device, group=None, pieces: int = 6,
                 timing: bool = False, quantum: int = 1024):
        self.engine, self.counts, self.N = engine, list(counts), int(N)
        self.group = group
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        assert len(self.counts) == self.world
        self.K = sum(self.counts)
        self.device = torch.device(device)
        self.bounds = range_bounds(self.N, pieces if self.world > 1 else 1, quantum)
        # receive buffer of the broadcast; the owner of gBest does not use it
        self.gbest = torch.zeros(self.N if self.world > 1 else 0, dtype=torch.float32, device=self.device)
        self.all_losses = torch.zeros(self.K, dtype=torch.float32, device=self.device)
        self.timing = bool(timing) and self.device.type == "cuda"
        self._events = []

    def _mark(self):
        if not self.timing:
            return None
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    def sync(self, local_losses: torch.Tensor, t_iter: int = 0, lam: float = 1.0) -> int:
        """local_losses: this rank's counts[rank] losses (tensor on self.device)."""
        e0 = self._mark()
        if self.world > 1 and len(set(self.counts)) == 1:
            # equal shards: one collective straight into the K-float buffer
            dist.all_gather_into_tensor(self.all_losses, local_losses.to(self.device, torch.float32).contiguous(),
                                        group=self.group)
            self.engine.set_losses(self.all_losses)
        elif self.world > 1:
            # unequal shards: equal-sized pieces (collectives want them), padded to the largest shard
            widest = max(self.counts)
            mine = torch.zeros(widest, dtype=torch.float32, device=self.device)
            mine[:self.counts[self.rank]] = local_losses.to(self.device, torch.float32)
            pieces = [torch.empty_like(mine) for _ in range(self.world)]
            dist.all_gather(pieces, mine, group=self.group)
            at = 0
            for piece, n in zip(pieces, self.counts):
                self.all_losses[at:at + n] = piece[:n]
                at += n
            self.engine.set_losses(self.all_losses)
        else:
            self.engine.set_losses(local_losses)    # one rank holds the whole swarm: nothing to gather
        g = self.engine.shard_select()              # the same on every rank
        e1 = self._mark()
        owner, row = owner_of(g, self.counts)
        # The owner sends its row as it stands and reads gBest from it in place.
        src = self.engine.row(row) if owner == self.rank else self.gbest
        works = []
        if self.world > 1:
            root = dist.get_global_rank(self.group, owner) if self.group else owner
            for a, b in self.bounds:
                works.append(dist.broadcast(src[a:b], src=root, group=self.group, async_op=True))
        em = None
        for i, (a, b) in enumerate(self.bounds):
            if works:
                works[i].wait()                     # range i has arrived (its sender: has left)
            if len(self.bounds) == 1:
                em = self._mark()                   # nothing overlaps: the exchange ends here
            self.engine.shard_update_range(src, a, b, t_iter, lam)
        e2 = self._mark()
        if self.timing:
            self._events.append((e0, e1, em, e2))
        return g

    def timings_ms(self) -> dict:
        """Mean device time per sync of the phases, over the syncs since the last
        call: losses + selection (with the host's read of g), then the gBest
        exchange with the updates it overlaps; with a single range (pieces = 1)
        nothing overlaps and exchange and update are also given separately."""
        if not self._events:
            return {"select_ms": None, "exchange_and_update_ms": None, "exchange_ms": None,
                    "update_ms": None, "syncs": 0}
        torch.cuda.synchronize(self.device)
        n = len(self._events)
        sel = sum(a.elapsed_time(b) for a, b, _, _ in self._events) / n
        both = sum(b.elapsed_time(d) for _, b, _, d in self._events) / n
        exch = upd = None                           # separable only when the sync used a single range
        if all(m is not None for _, _, m, _ in self._events):
            exch = sum(b.elapsed_time(m) for _, b, m, _ in self._events) / n
            upd = sum(m.elapsed_time(d) for _, _, m, d in self._events) / n
        self._events = []
        return {"select_ms": sel, "exchange_and_update_ms": both, "exchange_ms": exch, "update_ms": upd,
                "syncs": n}


def swarm_engine(swarm):
    """Adapter from a binding.Swarm created with k_first / K_total."""

    class _Engine:
        def set_losses(self, all_losses):
            swarm.set_losses(all_losses)

        def shard_select(self):
            return swarm.shard_select()

        def row(self, row):
            return swarm.x[row, :swarm.N]

        def shard_update_range(self, gbest, first, last, t_iter, lam):
            swarm.shard_update_range(gbest, first, last, t_iter, lam)

    return _Engine()
