"""Randomised parity: shapes, strides, misalignment, hyper-parameters, flags and
loss patterns drawn from a seeded generator; every case runs a few syncs on the
GPU and in the oracle and must agree bit for bit."""
import numpy as np
import pytest

from paper_2009_03816_b200 import binding

import gpu_util
from gpu_util import Pair

pytestmark = pytest.mark.gpu


def _case(rng):
    K = int(rng.choice([1, 2, 3, 5, 8, 31, 32, 33, 64, 65, 100]))
    N = int(rng.choice([1, 2, 3, 4, 5, 7, 31, 32, 33, 127, 128, 129, 255, 256, 257, 1000, 1023, 1024,
                        1025, 4095, 4097, 10_000, 33_333]))
    aligned = rng.random() < 0.6
    if aligned:
        ld, offset = (N + 3) // 4 * 4 + 4 * int(rng.integers(0, 3)), 0
    else:
        ld, offset = N + int(rng.integers(0, 4)), int(rng.integers(0, 4))
        if ld % 4 == 0 and offset == 0:
            offset = 1
    flags = int(rng.choice([0, binding.PSOPS_KEEP_GBEST, binding.PSOPS_GBEST_HISTORY]))
    m_max = float(rng.uniform(0.3, 1.1))
    m_min = float(rng.uniform(0.0, m_max))
    return dict(K=K, N=N, ld=ld, offset=offset, flags=flags, m_max=m_max, m_min=m_min,
                t_max=int(rng.integers(1, 1000)), c1=float(rng.uniform(0, 2.5)), c2=float(rng.uniform(0, 2.5)),
                seed=int(rng.integers(0, 1 << 63)) * 2 + int(rng.integers(0, 2)))


@pytest.mark.parametrize("block", range(8))
def test_random_cases(block):
    rng = np.random.default_rng(1000 + block)
    for _ in range(12):
        c = _case(rng)
        K, N = c["K"], c["N"]
        x = rng.standard_normal((K, N)).astype(np.float32) * np.float32(rng.choice([1e-3, 1.0, 50.0]))
        v = rng.standard_normal((K, N)).astype(np.float32) * np.float32(rng.choice([0.0, 1e-4, 1.0]))
        p = x.copy() if rng.random() < 0.5 else (x + rng.standard_normal((K, N))).astype(np.float32)
        pair = Pair(x, v, p, N, ld=c["ld"], offset=c["offset"], m_max=c["m_max"], m_min=c["m_min"],
                    t_max=c["t_max"], c1=c["c1"], c2=c["c2"], seed=c["seed"], flags=c["flags"])
        if c["flags"] & binding.PSOPS_GBEST_HISTORY:
            import oracle
            pair.ref = oracle.RefSwarm(x, v, p, m_max=c["m_max"], m_min=c["m_min"], t_max=c["t_max"],
                                       c1=c["c1"], c2=c["c2"], seed=c["seed"], history=True)
        for s in range(int(rng.integers(1, 5))):
            kind = rng.random()
            if kind < 0.3:
                loss = rng.integers(0, 3, size=K).astype(np.float32)           # ties
            elif kind < 0.4:
                loss = np.full(K, np.inf, np.float32)
            else:
                loss = rng.random(K).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 3))
            t = int(rng.integers(0, 2 * c["t_max"]))
            lam = float(rng.choice([1.0, 1.5, 7.0, 25.0]))
            pair.sync(loss, t, lam)
            pair.check_selection()
            pair.check_state(f"{c} s={s}")
        assert pair.inexact == 0, c
        pair.check_canaries(str(c))
        pair.close()
