"""Algorithm 1 end to end on the quadratic stand-in objective: PSO-PS, parameter
averaging and synchronous SGD side by side.

    python -m paper_2009_03816_b200.demo [--epochs 25] [--n 65536] ...

K workers start from the same weights (Algorithm 2) and minimise
f(w) = sum_j d_j (w_j - t_j)^2.  Worker k only sees its own shard of the data,
modelled as a shifted target t_k = t + sigma * xi_k, so its local gradient is
2 d (w - t_k).  Between synchronisations every worker takes plain gradient
steps ("else update w by SGD" in Algorithm 1); that local training is outside
the library and is done here with a few torch operations.  Everything the
paper's synchronisation stage does runs in the CUDA library through its C ABI:

  pso   every `step` iterations: fitness of every worker's weights on the
        device (psops_eval_quadratic), then one PSO-PS synchronisation
        (psops_sync: Algorithm 3, the pBest branch, Eq. 5-7) with Table II's
        settings: m from 0.9 to 0.3, c1 = 0.2, c2 = 0.9, lambda = epoch index
  pa    every `step` iterations: parameter averaging (psops_average,
        Section II-B steps 3-5)
  ssgd  every iteration: w <- w + (alpha / K) sum_k grad_k with alpha = -lr
        (psops_ssgd, Section II-B)

The result is one JSON object with, per method and epoch, the best and the mean
worker loss (f evaluated on the device).  An `observer` sees the weights before
and after every synchronisation, which is how the tests run the CPU oracle
beside the library.
"""
from __future__ import annotations

import argparse
import json
from dataclasses import asdict, dataclass

import numpy as np
import torch

from . import binding
from . import build as _build


@dataclass(frozen=True)
class DemoConfig:
    K: int = 8                   # workers = particles
    N: int = 65_536              # parameters
    epochs: int = 25             # Table II / Section IV: 25 epochs
    iters_per_epoch: int = 50
    step: int = 10               # iterations between synchronisations (Algorithm 1)
    lr: float = 0.05
    shard_sigma: float = 0.3     # how far a worker's shard pulls away from the common target
    seed: int = 7
    m_max: float = 0.9           # Table II
    m_min: float = 0.3
    c1: float = 0.2
    c2: float = 0.9

    @property
    def t_max(self) -> int:
        return self.epochs * self.iters_per_epoch

    @property
    def ld(self) -> int:
        return (self.N + 1023) // 1024 * 1024


def problem(cfg: DemoConfig, device):
    """(dvec, tvec, per-worker targets, common initial weights), seeded."""
    rng = np.random.default_rng([cfg.seed, 41])
    d = (0.5 + 1.5 * rng.random(cfg.N, dtype=np.float32)).astype(np.float32)
    t = rng.standard_normal(cfg.N, dtype=np.float32)
    shard_t = (t + np.float32(cfg.shard_sigma) * rng.standard_normal((cfg.K, cfg.N), dtype=np.float32))
    w0 = rng.standard_normal(cfg.N, dtype=np.float32)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return to(d), to(t), to(shard_t), to(w0)


class _Losses:
    """Fitness of the K rows on the device: attach the quadratic, evaluate,
    detach again (the sync that follows must not fuse the fitness of the NEW
    weights in: Algorithm 1 wants the losses of the weights as trained)."""

    def __init__(self, sw, d, t):
        self.sw, self.d, self.t = sw, d, t

    def evaluate(self) -> np.ndarray:
        self.sw.set_quadratic(self.d, self.t)
        self.sw.eval_quadratic()
        binding.psops_set_quadratic(self.sw.ctx, None, None)
        return self.sw.losses()


def run(method: str, cfg: DemoConfig = DemoConfig(), device="cuda:0", observer=None) -> dict:
    """Run one method for cfg.epochs epochs.  observer(event: dict) is called
    around every synchronisation with host copies of what went in and what came
    out (see the keys below)."""
    assert method in ("pso", "pa", "ssgd")
    _build.build_library()
    device = torch.device(device)
    d, t, shard_t, w0 = problem(cfg, device)
    N, ld, K = cfg.N, cfg.ld, cfg.K
    x = torch.zeros((K, ld), dtype=torch.float32, device=device)
    x[:, :N] = w0
    v = torch.zeros_like(x)
    p = x.clone()
    sw = binding.Swarm(x, v, p, N=N, m_max=cfg.m_max, m_min=cfg.m_min, t_max=cfg.t_max, c1=cfg.c1, c2=cfg.c2,
                       seed=cfg.seed, flags=binding.PSOPS_QUADRATIC)
    fitness = _Losses(sw, d, t)
    period = 1 if method == "ssgd" else cfg.step
    w = x[:, :N]                                     # the workers' weights, a view of the swarm's rows
    grad = torch.zeros((K, ld), dtype=torch.float32, device=device)
    curve_best, curve_mean, syncs = [], [], 0
    host = lambda tensor: tensor[:, :N].cpu().numpy()
    initial_loss = float(fitness.evaluate()[0])       # all workers start from the same weights
    for it in range(1, cfg.t_max + 1):
        epoch = 1 + (it - 1) // cfg.iters_per_epoch
        grad[:, :N] = 2.0 * d * (w - shard_t)        # each worker's gradient on its own shard
        if method == "ssgd":
            if observer:
                before = {"x": host(x), "grad": host(grad)}
            sw.ssgd(grad, -cfg.lr)
            syncs += 1
            if observer:
                observer({"method": method, "iteration": it, "alpha": -cfg.lr, **before, "x_after": host(x)})
        else:
            w -= cfg.lr * grad[:, :N]                # Algorithm 1: "update w by SGD"
            if it % period == 0:
                if method == "pa":
                    if observer:
                        before = {"x": host(x)}
                    sw.average()
                    if observer:
                        observer({"method": method, "iteration": it, **before, "x_after": host(x)})
                else:
                    losses = fitness.evaluate()
                    if observer:
                        before = {"x": host(x), "losses": losses.copy()}
                    sw.sync(it, float(epoch))         # lambda = epoch index (Table II)
                    if observer:
                        g, improved, pbest_loss = sw.info()
                        observer({"method": method, "iteration": it, "lambda": float(epoch), **before,
                                  "g": g, "improved": improved, "pbest_loss": pbest_loss,
                                  "x_after": host(x), "v_after": host(v), "p_after": host(p)})
                syncs += 1
        if it % cfg.iters_per_epoch == 0:
            losses = fitness.evaluate()
            curve_best.append(float(losses.min()))
            curve_mean.append(float(losses.mean()))
    torch.cuda.synchronize(device)
    sw.close()
    return {"method": method, "syncs": syncs, "initial_loss": initial_loss, "best_loss": curve_best,
            "mean_loss": curve_mean}


def main(argv=None) -> dict:
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    for name, default in asdict(DemoConfig()).items():
        ap.add_argument("--" + name.replace("_", "-").lower(), type=type(default), default=default)
    ap.add_argument("--device", default="cuda:0")
    args = vars(ap.parse_args(argv))
    device = args.pop("device")
    cfg = DemoConfig(**{k: args[k.lower()] for k in asdict(DemoConfig())})
    out = {"config": asdict(cfg), "objective": "f(w) = sum_j d_j (w_j - t_j)^2, d ~ U[0.5, 2], t ~ N(0, 1)",
           "methods": {}}
    for method in ("pso", "pa", "ssgd"):
        out["methods"][method] = run(method, cfg, device)
    print(json.dumps(out))
    return out


if __name__ == "__main__":
    main()
