"""Algorithm 1 end to end on the quadratic stand-in objective (the demo module:
local gradient steps between synchronisations, PSO-PS / parameter averaging /
SSGD through the library) with the CPU oracle run beside the library at every
synchronisation: it is handed the same post-local-step weights and must
produce the same selection and the same new state."""
import json

import numpy as np
import pytest

import oracle
from paper_2009_03816_b200 import demo

from gpu_util import NTHREADS, assert_close

pytestmark = pytest.mark.gpu

CFG = demo.DemoConfig(K=8, N=20_003, epochs=5, iters_per_epoch=20, step=10, seed=3)


def _problem_on_host(cfg):
    d, t, shard_t, w0 = demo.problem(cfg, "cuda:0")
    return d.cpu().numpy(), t.cpu().numpy(), w0.cpu().numpy()


def test_pso_arm_with_the_oracle_in_the_loop():
    cfg = CFG
    d, t, w0 = _problem_on_host(cfg)
    start = np.tile(w0, (cfg.K, 1))
    ref = oracle.RefSwarm(start, np.zeros_like(start), start, m_max=cfg.m_max, m_min=cfg.m_min,
                          t_max=cfg.t_max, c1=cfg.c1, c2=cfg.c2, seed=cfg.seed, nthreads=NTHREADS)
    seen = []

    def observer(ev):
        # local training happened outside the library and outside the oracle:
        # the oracle takes the weights as trained, everything else is its own
        ref.x[:] = ev["x"]
        loss = oracle.quadratic_losses(ref.x, d, t, nthreads=NTHREADS)
        assert np.array_equal(loss.view(np.uint32), ev["losses"].view(np.uint32)), ev["iteration"]
        ref.sync(loss, ev["iteration"], ev["lambda"])
        assert ev["g"] == ref.g and np.array_equal(ev["improved"], ref.improved), ev["iteration"]
        assert np.array_equal(ev["pbest_loss"].view(np.uint32), ref.pbest_loss.view(np.uint32))
        inexact = 0
        for got, want, name in ((ev["x_after"], ref.x, "x"), (ev["v_after"], ref.v, "v"), (ev["p_after"], ref.p, "pbest")):
            inexact += assert_close(got, want, f"sync at iteration {ev['iteration']} {name}")
        assert inexact == 0
        seen.append(ev["iteration"])

    out = demo.run("pso", cfg, observer=observer)
    assert seen == list(range(cfg.step, cfg.t_max + 1, cfg.step)) and out["syncs"] == len(seen)
    assert len(out["best_loss"]) == cfg.epochs
    assert out["best_loss"][-1] < 0.05 * out["initial_loss"]


def test_pa_and_ssgd_arms_with_the_oracle_in_the_loop():
    cfg = CFG
    checked = {"pa": 0, "ssgd": 0}

    def observer(ev):
        want = ev["x"].copy()
        if ev["method"] == "pa":
            oracle.average(want, nthreads=NTHREADS)
        else:
            oracle.ssgd(want, ev["grad"], ev["alpha"], nthreads=NTHREADS)
        assert np.array_equal(ev["x_after"].view(np.uint32), want.view(np.uint32)), (ev["method"], ev["iteration"])
        checked[ev["method"]] += 1

    pa = demo.run("pa", cfg, observer=observer)
    ssgd = demo.run("ssgd", cfg, observer=observer)
    assert checked == {"pa": cfg.t_max // cfg.step, "ssgd": cfg.t_max}
    for out in (pa, ssgd):
        assert out["best_loss"][-1] < 0.05 * out["initial_loss"]
    # averaging and gradient averaging cancel the shards' pull: they end far below one worker's shard noise
    shard_floor = cfg.shard_sigma ** 2 * 1.25 * cfg.N
    assert pa["best_loss"][-1] < 0.5 * shard_floor and ssgd["best_loss"][-1] < 0.5 * shard_floor


def test_demo_main_prints_three_curves(capsys):
    out = demo.main(["--epochs", "3", "--iters-per-epoch", "10", "--n", "4099", "--k", "4"])
    printed = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert printed == out and set(out["methods"]) == {"pso", "pa", "ssgd"}
    for m in out["methods"].values():
        assert len(m["best_loss"]) == 3 and all(np.isfinite(m["best_loss"]))
        assert m["best_loss"][-1] < m["initial_loss"]
