"""Algorithm 1 end to end on a toy problem: K workers take local gradient steps
on their own noisy shard of a quadratic objective (plain torch ops stand in for
local training, which is not part of the library) and synchronise every `step`
iterations with PSO-PS, with parameter averaging, or -- at step = 1 -- with
SSGD.  A sanity check that the three synchronisation methods of Section II-B /
Section III drive the same objective down when called through the library."""
import numpy as np
import pytest
import torch

from paper_2009_03816_b200 import binding

import gpu_util

pytestmark = pytest.mark.gpu

K, N, STEP, ITERS_PER_EPOCH, EPOCHS, ETA = 8, 50_000, 10, 40, 5, 0.05


def _problem(seed=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    d = torch.rand(N, device="cuda", generator=g) * 1.5 + 0.5
    t = torch.randn(N, device="cuda", generator=g)
    shard_t = t + 0.3 * torch.randn((K, N), device="cuda", generator=g)       # each worker's data differs
    w0 = torch.randn(N, device="cuda", generator=g).repeat(K, 1).contiguous()  # Algorithm 1: same initial weights
    return d, t, shard_t, w0


def _global_loss(w, d, t):
    return (d * (w - t) ** 2).sum(dim=1)


def _local_grad(w, d, shard_t):
    return 2.0 * d * (w - shard_t)


def _run(method):
    gpu_util.ensure_library()
    d, t, shard_t, w0 = _problem()
    x, v, p = w0.clone(), torch.zeros_like(w0), w0.clone()
    t_max = EPOCHS * ITERS_PER_EPOCH
    sw = binding.Swarm(x, v, p, m_max=0.9, m_min=0.3, t_max=t_max, c1=0.2, c2=0.9, seed=11,
                       flags=binding.PSOPS_QUADRATIC)
    first = float(_global_loss(x, d, t).min())
    period = 1 if method == "ssgd" else STEP
    for it in range(1, t_max + 1):
        grad = _local_grad(x, d, shard_t)
        if method == "ssgd":
            sw.ssgd(grad, -ETA)                                   # w <- w + (alpha / n) sum grad_k, alpha = -eta
            continue
        x -= ETA * grad                                           # Algorithm 1: "update w by SGD"
        if it % period == 0:
            if method == "pa":
                sw.average()
            else:
                sw.set_quadratic(d, t)
                sw.eval_quadratic()                               # fitness = loss of the current weights
                binding.psops_set_quadratic(sw.ctx, None, None)   # detach: the losses of the weights as
                sw.sync(it, 1.0 + (it - 1) // ITERS_PER_EPOCH)    # trained are wanted, not those after the sync
    torch.cuda.synchronize()
    last = float(_global_loss(x, d, t).min())
    spread = float((x - x.mean(dim=0)).abs().max())
    sw.close()
    return first, last, spread


def test_three_synchronisation_methods_reduce_the_objective():
    res = {m: _run(m) for m in ("pso", "pa", "ssgd")}
    noise_floor = 0.3 ** 2 * 1.25 * N            # a worker that fits only its own shard ends near here
    for m, (first, last, spread) in res.items():
        assert last < 0.05 * first, (m, first, last)
        assert np.isfinite(last)
    # averaging and gradient averaging cancel most of the shard noise; PSO-PS keeps
    # the workers apart (it is a search, not a consensus) but must not be worse than
    # a worker left alone with its shard
    assert res["pa"][1] < 0.5 * noise_floor and res["ssgd"][1] < 0.5 * noise_floor
    assert res["pso"][1] < 1.5 * noise_floor
    assert res["ssgd"][2] == 0.0                 # SSGD hands every worker the same weights
