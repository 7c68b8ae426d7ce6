"""Seeded synthetic inputs for the PSO-PS synchronisation stage.

The paper trains LeNet on MNIST and a ResNet on CIFAR10 with n = 4..16
workers; neither the datasets nor the models are used here.  These
generators only take the *shapes* of those workloads (flat parameter-vector
lengths, worker counts) and fill them with seeded random numbers.  They hold
no arithmetic of the method: the same arrays are handed to the CUDA library
and, separately, to whatever checks it.

Every row of every array has its own stream
``numpy.random.default_rng([seed, tag, row])`` so that any row (or a sample of
its columns) can be regenerated without materialising the rest.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np

_TAG_X, _TAG_V, _TAG_LOSS, _TAG_D, _TAG_T = 11, 12, 13, 14, 15


@dataclass(frozen=True)
class Workload:
    name: str
    K: int                 # particles = workers
    N: int                 # elements per particle
    S: int                 # synchronisation steps
    omega: float           # constant inertia (m_max == m_min)
    c1: float
    c2: float
    seed: int
    sigma_x: float
    sigma_v: float         # 0 -> v starts at zero
    loss_lo: float = 0.0
    loss_hi: float = 1.0
    ties: bool = False     # deliberate equal losses (see losses())
    quadratic: bool = False  # fitness evaluated on device, no loss table
    lam: float = 1.0
    note: str = ""
    # Table II style schedules (all zero / None: constant inertia omega, constant lambda)
    m_min: float | None = None   # Eq. 5 lower inertia; m_max is `omega`
    sync_period: int = 0         # `step` of Algorithm 1: training iterations between syncs
    iters_per_epoch: int = 0     # training-set size / batch size
    epochs: int = 0              # lambda = epoch index 1..epochs; t_max = epochs * iters_per_epoch

    @property
    def ld(self) -> int:
        """Row stride in elements: N rounded up to a multiple of 1024, so that
        every row starts on a 4-KiB boundary.  16-byte alignment is what the
        128-bit kernels need; the 4-KiB pitch is worth a further ~4 % of HBM
        bandwidth on B200 (measured) for at most 4 KiB of padding per row."""
        return (self.N + 1023) // 1024 * 1024

    @property
    def m_max(self) -> float:
        return self.omega

    @property
    def m_lo(self) -> float:
        return self.omega if self.m_min is None else self.m_min

    @property
    def t_max(self) -> int:
        return self.epochs * self.iters_per_epoch if self.epochs else 1

    def schedule(self, s: int) -> tuple[int, float]:
        """(t_iter, lambda) of sync s: Algorithm 1 syncs whenever t % step == 0,
        t counting training iterations from 1; lambda is the 1-based epoch."""
        if not self.sync_period:
            return 0, self.lam
        t = (s + 1) * self.sync_period
        return t, float(min(self.epochs, 1 + (t - 1) // self.iters_per_epoch))

    def with_particles(self, K: int) -> "Workload":
        """Same recipe with another number of rows (e.g. the rows one shard holds)."""
        return replace(self, K=int(K))

    def scaled(self, N: int, S: int | None = None) -> "Workload":
        """Same recipe at another vector length (parity cases that a CPU
        check finishes in seconds)."""
        return replace(self, N=int(N), S=self.S if S is None else int(S),
                       name=f"{self.name}@N={int(N)}")


CONFIGS = {
    "cfg1": Workload("cfg1", K=4, N=61_706, S=10, omega=0.7, c1=1.5, c2=1.5,
                     seed=1, sigma_x=0.05, sigma_v=0.0, loss_lo=0.1, loss_hi=2.5,
                     note="LeNet-5-sized flat vector"),
    "cfg2": Workload("cfg2", K=8, N=1_250_000, S=50, omega=0.9, c1=2.0, c2=2.0,
                     seed=2, sigma_x=0.02, sigma_v=1e-3, loss_lo=0.5, loss_hi=2.3,
                     note="small CNN for 32x32x3 inputs"),
    "cfg3": Workload("cfg3", K=16, N=11_173_962, S=100, omega=0.7, c1=1.5, c2=1.5,
                     seed=3, sigma_x=0.01, sigma_v=0.0, loss_lo=0.2, loss_hi=2.3,
                     ties=True, note="ResNet-18-sized"),
    "cfg4": Workload("cfg4", K=32, N=25_557_032, S=100, omega=0.6, c1=1.8, c2=1.8,
                     seed=4, sigma_x=0.01, sigma_v=1e-4, loss_lo=0.1, loss_hi=2.5,
                     note="ResNet-50-sized"),
    "cfg5": Workload("cfg5", K=8, N=50_000_000, S=200, omega=0.7, c1=1.5, c2=1.5,
                     seed=5, sigma_x=1.0, sigma_v=0.0, quadratic=True,
                     note="quadratic fitness evaluated on device"),
    # The paper's own settings (Table II: m 0.9 -> 0.3, c1 0.2, c2 0.9, lambda = epoch) on its
    # LeNet/MNIST schedule: 60,000 samples / batch 256 = 234 iterations per epoch, 25 epochs,
    # a sync every 10 iterations -> 585 syncs.  Only shapes and the schedule are used.
    "cfg6": Workload("cfg6", K=8, N=61_706, S=585, omega=0.9, m_min=0.3, c1=0.2, c2=0.9,
                     seed=6, sigma_x=0.05, sigma_v=0.0, loss_lo=0.1, loss_hi=2.5,
                     sync_period=10, iters_per_epoch=234, epochs=25,
                     note="Table II schedule on a LeNet-5-sized vector"),
}


def _rng(w: Workload, tag: int, row: int = 0) -> np.random.Generator:
    return np.random.default_rng([w.seed, tag, row])


def x_row(w: Workload, k: int) -> np.ndarray:
    """Initial weights of particle k: N(0, sigma_x), fp32."""
    r = _rng(w, _TAG_X, k).standard_normal(w.N, dtype=np.float32)
    r *= np.float32(w.sigma_x)
    return r


def v_row(w: Workload, k: int) -> np.ndarray:
    """Initial velocity of particle k: zeros or N(0, sigma_v), fp32."""
    if w.sigma_v == 0.0:
        return np.zeros(w.N, dtype=np.float32)
    r = _rng(w, _TAG_V, k).standard_normal(w.N, dtype=np.float32)
    r *= np.float32(w.sigma_v)
    return r


def state(w: Workload):
    """(x, v, pbest) as three (K, ld) fp32 arrays, padding zero, pbest = x."""
    x = np.zeros((w.K, w.ld), dtype=np.float32)
    v = np.zeros((w.K, w.ld), dtype=np.float32)
    for k in range(w.K):
        x[k, :w.N] = x_row(w, k)
        v[k, :w.N] = v_row(w, k)
    return x, v, x.copy()


def quadratic_vectors(w: Workload):
    """(dvec ~ U[0.5, 2], tvec ~ N(0, 1)) of the quadratic stand-in fitness."""
    d = _rng(w, _TAG_D).random(w.N, dtype=np.float32)
    d = (np.float32(0.5) + np.float32(1.5) * d).astype(np.float32)
    t = _rng(w, _TAG_T).standard_normal(w.N, dtype=np.float32)
    return d, t


def losses(w: Workload) -> np.ndarray:
    """(S, K) fp32 table of per-sync losses ~ U[loss_lo, loss_hi].

    With ``ties`` set, each step with probability 1/2 the minimum is copied to
    one other random index (lower and higher indices both occur), and with
    probability 1/4 one particle is handed the smallest loss it has been given
    so far again (an equal loss, which must not count as an improvement).
    """
    rng = _rng(w, _TAG_LOSS)
    tab = rng.random((w.S, w.K), dtype=np.float32)
    tab = (np.float32(w.loss_lo)
           + np.float32(w.loss_hi - w.loss_lo) * tab).astype(np.float32)
    if w.ties and w.K > 1:
        seen_min = np.full(w.K, np.inf, dtype=np.float32)
        for s in range(w.S):
            row = tab[s]
            coin_tie, coin_repeat = rng.random(), rng.random()
            j, i = int(rng.integers(w.K - 1)), int(rng.integers(w.K))
            if s > 0 and coin_repeat < 0.25:
                row[i] = seen_min[i]
            if coin_tie < 0.5:
                a = int(np.argmin(row))
                row[(a + 1 + j) % w.K] = row[a]
            seen_min = np.minimum(seen_min, row)
    return tab


def sample_columns(N: int, count: int, seed: int) -> np.ndarray:
    """Sorted element indices for spot checks at full size: the first and last
    few elements (vector head, ragged tail) plus a seeded random draw."""
    edge = np.concatenate([np.arange(min(8, N)), np.arange(max(0, N - 8), N)])
    rnd = np.random.default_rng([seed, 99]).integers(0, N, size=max(0, count))
    return np.unique(np.concatenate([edge, rnd]).astype(np.int64))


def sample_columns_dense(N: int, count: int, seed: int, block: int = 1024) -> np.ndarray:
    """A larger sample for full-size checks: `count` seeded random elements,
    plus one element of every residue modulo `block` (the elements one thread
    block of the update kernel covers) in a seeded random block, plus the first
    and last element of the first, a middle and the last block, plus the
    vector's head and ragged tail."""
    rng = np.random.default_rng([seed, 98])
    blocks = (N + block - 1) // block
    residues = np.arange(block, dtype=np.int64) + block * rng.integers(0, max(1, blocks - 1), size=block)
    edges = []
    for b in (0, blocks // 2, blocks - 1):
        edges += [b * block, min(N, (b + 1) * block) - 1]
    head_tail = np.concatenate([np.arange(min(8, N)), np.arange(max(0, N - 8), N)])
    rnd = rng.integers(0, N, size=max(0, count))
    cols = np.concatenate([residues, np.asarray(edges, dtype=np.int64), head_tail, rnd]).astype(np.int64)
    return np.unique(cols[(cols >= 0) & (cols < N)])
