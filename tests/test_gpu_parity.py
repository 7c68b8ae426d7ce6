"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on
the same seeded inputs -- selection bit-exact, x / v / pbest within 1e-6
relative after every sync, free-running (the GPU state is never refreshed from
the oracle)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2009_03816_b200 import binding, workloads
from paper_2009_03816_b200.binding import (PSOPS_GBEST, PSOPS_KEEP_GBEST, PSOPS_PBEST,
                                           PSOPS_QUADRATIC, PSOPS_SEPARATE_SELECT, PSOPS_V, PSOPS_X)

import gpu_util
from gpu_util import NTHREADS, Pair, assert_close

pytestmark = pytest.mark.gpu


def _swarm(K, N, seed, sv=0.1):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((K, N)).astype(np.float32)
    v = (sv * rng.standard_normal((K, N))).astype(np.float32)
    p = (x + 0.5 * rng.standard_normal((K, N))).astype(np.float32)
    return x, v, p


# ---------------------------------------------------------------------------
# Small shapes: several tiles, ragged tails, both kernels variants.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("N", [1, 2, 3, 5, 127, 128, 129, 1000, 4099])
@pytest.mark.parametrize("K,separate", [(1, False), (2, False), (3, False), (5, False), (8, False), (16, False),
                                        (32, False), (1, True), (2, True), (3, True), (8, True), (32, True),
                                        (33, True)])
def test_small_shapes_vector_path(K, N, separate):
    """Up to 8 particles a small sync is one launch that selects and updates
    (four particles in flight up to K = 4, eight beyond); PSOPS_SEPARATE_SELECT
    runs the selection kernel first; 9 or more particles on so few elements
    have their rows split over more blocks (a gBest snapshot that up to
    32 particles also selects, then the update).  All must follow the oracle bit for bit."""
    x, v, p = _swarm(K, N, 100 * K + N)
    pair = Pair(x, v, p, N, m_max=0.9, m_min=0.3, t_max=10, c1=0.2, c2=0.9, seed=K * 7919 + N,
                flags=PSOPS_SEPARATE_SELECT if separate else 0)
    rng = np.random.default_rng(N)
    for s in range(4):
        pair.sync(rng.random(K).astype(np.float32), t=3 * s, lam=1.0 + s)
        pair.check_selection()
        pair.check_state(f"K={K} N={N} s={s}")
    pair.check_canaries()
    assert pair.inexact == 0          # same rounding sequence on both sides
    # per sync: 1 launch (single-launch form), 2 (selection kernel + update, or selecting snapshot + row-split
    # update), 3 (selection, snapshot, row-split update)
    per_sync = 3 if (K > 32 or (K >= 9 and separate)) else 2 if (K >= 9 or separate) else 1
    assert pair.gpu.launches == 4 * per_sync
    pair.close()


@pytest.mark.parametrize("N,ld,offset", [(5, 5, 0), (129, 131, 0), (1000, 1000, 1), (1003, 1003, 3),
                                         (4096, 4096, 2), (777, 780, 1)])
@pytest.mark.parametrize("K", [1, 4, 33])
def test_small_shapes_scalar_path(K, N, ld, offset):
    x, v, p = _swarm(K, N, 3 * K + N)
    pair = Pair(x, v, p, N, ld=ld, offset=offset, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=N)
    rng = np.random.default_rng(K)
    for s in range(3):
        pair.sync(rng.random(K).astype(np.float32))
        pair.check_selection()
        pair.check_state(f"K={K} N={N} ld={ld} off={offset} s={s}")
    pair.check_canaries()
    assert pair.inexact == 0
    pair.close()


def test_many_particles():
    K, N = binding.PSOPS_MAX_K, 260
    x, v, p = _swarm(K, N, 5)
    pair = Pair(x, v, p, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=11)
    rng = np.random.default_rng(2)
    for s in range(3):
        loss = rng.integers(0, 50, size=K).astype(np.float32)      # many ties
        pair.sync(loss)
        pair.check_selection()
    pair.check_state("K=1024")
    pair.check_canaries()
    pair.close()


# ---------------------------------------------------------------------------
# Selection edge cases through the device kernel.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K", [7, 8, 12, 20, 40])     # selection inside the update launch (K <= 8) / selection kernel
def test_selection_ties_nan_inf_on_device(K):
    N = 64
    x, v, p = _swarm(K, N, 9)
    pair = Pair(x, v, p, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=3)
    rng = np.random.default_rng(1)
    cases = []
    for _ in range(20):
        loss = rng.integers(0, 3, size=K).astype(np.float32)
        cases.append(loss)
    cases.append(np.full(K, np.inf, np.float32))
    cases.append(np.where(np.arange(K) == K - 3, -0.0, 0.0).astype(np.float32))
    for loss in cases:
        pair.sync(loss)
        pair.check_selection()
    # device-side NaN losses (the host path refuses them): they never win
    dl = np.full(K, np.nan, np.float32)
    dl[K - 5] = 5.0
    dl[K - 4] = 5.0
    dev = torch.from_numpy(dl).cuda()
    pair.gpu.set_losses(dev)
    pair.gpu.sync()
    pair.ref.sync(dl)
    pair.check_selection()
    assert pair.ref.g == K - 5
    dev = torch.from_numpy(np.full(K, np.nan, np.float32)).cuda()
    pair.gpu.set_losses(dev)
    pair.gpu.sync()
    pair.ref.sync(np.full(K, np.nan, np.float32))
    pair.check_selection()
    assert pair.ref.g == 0
    pair.close()


@pytest.mark.parametrize("K", [5, 13])                 # 13: rows split into groups, gBest read from a snapshot
@pytest.mark.parametrize("g", [0, 1, 2, 3, 4])
def test_gbest_row_is_read_before_it_is_overwritten(g, K):
    N = 10_007
    g = g if K == 5 else 3 * g                           # 0, 3, 6, 9, 12: a row of every group
    x, v, p = _swarm(K, N, 77)
    pair = Pair(x, v, p, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=g, flags=PSOPS_KEEP_GBEST)
    loss = np.full(K, 2.0, np.float32)
    loss[g] = 1.0
    pair.sync(loss, want_gbest=True)
    pair.check_selection()
    assert pair.ref.g == g
    pair.check_state(f"g={g}")
    got = pair.gpu.row(PSOPS_GBEST)
    assert np.array_equal(got, x[g]) and np.array_equal(got, pair.ref.gbest)
    pair.close()


# ---------------------------------------------------------------------------
# The five workload recipes.
# ---------------------------------------------------------------------------
def _run_workload(w, every=1):
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    pair = Pair(x, v, p, w.N, ld=w.ld, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)
    for s in range(w.S):
        pair.sync(table[s], 0, w.lam)
        pair.check_selection()
        if s % every == 0 or s == w.S - 1:
            pair.check_state(f"{w.name} s={s}")
    pair.check_canaries(w.name)
    inexact = pair.inexact
    pair.close()
    return inexact


def test_cfg1_full():
    assert _run_workload(workloads.CONFIGS["cfg1"]) == 0


def test_cfg2_full():
    # omega=0.9, c=2.0 is outside PSO's stability region: trajectories amplify
    # any rounding difference, so this only passes with identical rounding.
    assert _run_workload(workloads.CONFIGS["cfg2"], every=7) == 0


@pytest.mark.parametrize("N", [500_003, 900_001, 1_600_002, 2_700_001])
def test_cfg2_recipe_across_the_cache_policies(N):
    """The update kernel keeps as many of the arrays x, v, pbest in L2 as fit in
    about half of it and streams the rest: with K = 8 these lengths give arrays
    of 16, 29, 51 and 86 MB, i.e. all three, two, one and none kept (on a GPU
    with 126 MB of L2).  The results must not depend on the choice."""
    w = workloads.CONFIGS["cfg2"].scaled(N=N, S=6)
    assert _run_workload(w, every=2) == 0


def test_cfg3_scaled_with_ties():
    w = workloads.CONFIGS["cfg3"].scaled(N=300_002)
    assert w.N % 4 == 2 and w.ld == 300_032          # ragged last quad, padded pitch
    assert _run_workload(w, every=9) == 0


def test_cfg4_scaled():
    assert _run_workload(workloads.CONFIGS["cfg4"].scaled(N=131_072 + 40, S=30), every=5) == 0


def _run_sampled(w, count):
    """Full-size run on the GPU in the launch configuration the benchmark times
    (device-resident loss table); the oracle follows a sample of columns (every
    element is independent of the others once the losses are given): `count`
    random ones, every residue of the element index modulo a thread block's
    1024 elements, block edges, the vector's head and ragged tail."""
    gpu_util.ensure_library()
    cols = workloads.sample_columns_dense(w.N, count, w.seed)
    assert cols.size >= count * 0.95 and set((cols % 1024).tolist()) == set(range(1024))
    dev = torch.device("cuda:0")
    dx = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    dv = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    xs = np.empty((w.K, cols.size), np.float32)
    vs = np.empty((w.K, cols.size), np.float32)
    for k in range(w.K):
        row = workloads.x_row(w, k)
        xs[k] = row[cols]
        dx[k, :w.N] = torch.from_numpy(row).to(dev)
        row = workloads.v_row(w, k)
        vs[k] = row[cols]
        dv[k, :w.N] = torch.from_numpy(row).to(dev)
    dp = dx.clone()
    table = workloads.losses(w)
    gpu = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)
    ref = oracle.RefSwarm(xs, vs, xs, m_max=w.omega, m_min=w.omega, t_max=1, c1=w.c1, c2=w.c2,
                          seed=w.seed, elem_index=cols, nthreads=NTHREADS)
    dtable = torch.from_numpy(table).to(dev)
    dcols = torch.from_numpy(cols).to(dev)
    inexact = 0
    for s in range(w.S):
        gpu.set_losses(dtable[s])                 # device-resident losses, as the benchmark does
        gpu.sync(0, w.lam)
        ref.sync(table[s], 0, w.lam)
        g, improved, pl = gpu.info()
        assert g == ref.g and np.array_equal(improved, ref.improved)
        assert np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32))
        if s % 10 == 0 or s == w.S - 1:
            for name, t, want in (("x", dx, ref.x), ("v", dv, ref.v), ("pbest", dp, ref.p)):
                got = t[:, dcols].cpu().numpy()
                inexact += assert_close(got, want, f"{w.name} s={s} {name}")
    assert torch.all(dx[:, w.N:] == 0) and torch.all(dv[:, w.N:] == 0) and torch.all(dp[:, w.N:] == 0)
    gpu.close()
    return inexact


def test_cfg3_full_size_sampled():
    assert _run_sampled(workloads.CONFIGS["cfg3"], 200_000) == 0


def test_cfg4_full_size_sampled():
    w = workloads.CONFIGS["cfg4"]
    assert workloads.sample_columns_dense(w.N, 1_050_000, w.seed).size >= 1_000_000
    assert _run_sampled(w, 1_050_000) == 0


def _run_whole_swarm(w, syncs, checkpoints):
    """Full size on both sides: the oracle carries the whole swarm (all host
    cores), selection is compared after every sync and EVERY element of x, v
    and pbest at the checkpoints and after the last sync.  Elements never
    interact, so a wrong element at any sync is still wrong at the end."""
    gpu_util.ensure_library()
    dev = torch.device("cuda:0")
    x, v, p = workloads.state(w)
    dx, dv = torch.from_numpy(x).to(dev), torch.from_numpy(v).to(dev)
    dp = dx.clone()
    ref = oracle.RefSwarm(x[:, :w.N], v[:, :w.N], p[:, :w.N], m_max=w.omega, m_min=w.omega, t_max=1,
                          c1=w.c1, c2=w.c2, seed=w.seed, nthreads=NTHREADS)
    del x, v, p
    table = workloads.losses(w)
    dtable = torch.from_numpy(table).to(dev)
    gpu = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)
    inexact = 0
    for s in range(syncs):
        gpu.set_losses(dtable[s])
        gpu.sync(0, w.lam)
        ref.sync(table[s], 0, w.lam)
        g, improved, pl = gpu.info()
        assert g == ref.g and np.array_equal(improved, ref.improved), s
        assert np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32)), s
        if s in checkpoints or s == syncs - 1:
            for name, t, want in (("x", dx, ref.x), ("v", dv, ref.v), ("pbest", dp, ref.p)):
                inexact += gpu_util.device_compare(t[:, :w.N], want, f"{w.name} s={s} {name}")
    assert torch.all(dx[:, w.N:] == 0) and torch.all(dv[:, w.N:] == 0) and torch.all(dp[:, w.N:] == 0)
    gpu.close()
    return inexact


def test_cfg3_full_size_whole_swarm_all_syncs():
    w = workloads.CONFIGS["cfg3"]
    assert _run_whole_swarm(w, w.S, checkpoints=(0, 9, 49)) == 0


def test_cfg4_full_size_whole_swarm_first_syncs():
    import psutil
    if psutil.virtual_memory().available < (40 << 30):
        pytest.skip("the oracle's copy of the 9.8 GB swarm plus the generator's needs about 30 GB of host memory")
    assert _run_whole_swarm(workloads.CONFIGS["cfg4"], 3, checkpoints=(0,)) == 0


# ---------------------------------------------------------------------------
# Quadratic fitness on the device (stand-alone and fused into the update).
# ---------------------------------------------------------------------------
def _quadratic_pair(w, flags=PSOPS_QUADRATIC):
    x, v, p = workloads.state(w)
    d, t = workloads.quadratic_vectors(w)
    pair = Pair(x, v, p, w.N, ld=w.ld, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed,
                flags=flags)
    dd, dt = torch.from_numpy(d).cuda(), torch.from_numpy(t).cuda()
    pair.gpu.set_quadratic(dd, dt)
    return pair, d, t


@pytest.mark.parametrize("N", [1, 3, 127, 128, 129, 4096 + 5, 131_072 * 3 + 77])
def test_quadratic_fitness_standalone_bit_exact(N):
    w = workloads.CONFIGS["cfg5"].scaled(N=N)
    pair, d, t = _quadratic_pair(w)
    pair.gpu.eval_quadratic()
    got = pair.gpu.losses()
    want = oracle.quadratic_losses(pair.ref.x, d, t, nthreads=NTHREADS)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    pair.close()


def _fitness_order_cases():
    import golden_cases
    return golden_cases.fitness_order_cases()


@pytest.mark.parametrize("case", _fitness_order_cases(), ids=lambda c: c[0])
def test_quadratic_fitness_hand_worked_order_on_device(case):
    """The hand-worked cancellation cases that fix the summation order and the
    term rounding, through the stand-alone fitness kernels and through the
    fitness fused into the update (pure inertia, v = 0: the new weights equal
    the old ones exactly, so the fused pass sees the same rows)."""
    name, w, d, t, want = case
    n = w.size
    x = np.stack([w, t, w])                              # row 1 sits at the minimiser: fitness 0
    zeros = np.zeros_like(x)
    pair = Pair(x, zeros, x, n, m_max=1.0, m_min=1.0, c1=0.0, c2=0.0, seed=1, flags=PSOPS_QUADRATIC)
    dd, dt = torch.from_numpy(d).cuda(), torch.from_numpy(t).cuda()
    pair.gpu.set_quadratic(dd, dt)
    pair.gpu.eval_quadratic()
    got = pair.gpu.losses()
    assert got[0].view(np.uint32) == want.view(np.uint32), (name, float(got[0]), float(want))
    assert got[2].view(np.uint32) == want.view(np.uint32) and got[1] == 0.0
    pair.gpu.sync()                                      # x' = x + 1 * 0 exactly; losses of x' from the fused pass
    fused = pair.gpu.losses()
    assert np.array_equal(pair.dx.host(), x)
    assert fused[0].view(np.uint32) == want.view(np.uint32), (name, float(fused[0]), float(want))
    assert fused[2].view(np.uint32) == want.view(np.uint32) and fused[1] == 0.0
    pair.close()


def test_cfg5_scaled_fused_fitness_every_step():
    w = workloads.CONFIGS["cfg5"].scaled(N=1_000_003, S=200)
    pair, d, t = _quadratic_pair(w)
    pair.gpu.eval_quadratic()
    loss = oracle.quadratic_losses(pair.ref.x, d, t, nthreads=NTHREADS)
    best = []
    for s in range(w.S):
        assert np.array_equal(pair.gpu.losses().view(np.uint32), loss.view(np.uint32)), s
        pair.gpu.sync(0, w.lam)                   # losses come from the device
        pair.ref.sync(loss, 0, w.lam)
        pair.check_selection()
        loss = oracle.quadratic_losses(pair.ref.x, d, t, nthreads=NTHREADS)
        if s % 20 == 0 or s == w.S - 1:
            pair.check_state(f"{w.name} s={s}")
        best.append(float(pair.ref.pbest_loss.min()))
    assert np.array_equal(pair.gpu.losses().view(np.uint32), loss.view(np.uint32))
    assert all(a >= b for a, b in zip(best, best[1:]))
    assert pair.inexact == 0
    pair.check_canaries()
    pair.close()


def test_cfg5_scalar_path_fused_fitness():
    w = workloads.CONFIGS["cfg5"].scaled(N=70_001, S=5)
    x, v, p = workloads.state(w)
    d, t = workloads.quadratic_vectors(w)
    pair = Pair(x, v, p, w.N, ld=w.N, offset=1, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                seed=w.seed, flags=PSOPS_QUADRATIC)
    dd, dt = torch.from_numpy(d).cuda(), torch.from_numpy(t).cuda()
    pair.gpu.set_quadratic(dd, dt)
    pair.gpu.eval_quadratic()
    loss = oracle.quadratic_losses(pair.ref.x, d, t)
    for s in range(w.S):
        assert np.array_equal(pair.gpu.losses().view(np.uint32), loss.view(np.uint32))
        pair.gpu.sync()
        pair.ref.sync(loss)
        pair.check_selection()
        pair.check_state(f"s={s}")
        loss = oracle.quadratic_losses(pair.ref.x, d, t)
    pair.check_canaries()
    pair.close()


def test_cfg5_full_size(syncs=None):
    """Full 50 M-element vectors, fitness fused into the update; the oracle
    runs the whole swarm on all host cores.  All 200 syncs of the recipe by
    default (PSOPS_CFG5_SYNCS shortens the run for a quick look): losses bit-exact
    and selection identical after every sync, every element of x, v, pbest at
    three checkpoints and at the end."""
    syncs = int(os.environ.get("PSOPS_CFG5_SYNCS", "200")) if syncs is None else syncs
    w = workloads.CONFIGS["cfg5"]
    gpu_util.ensure_library()
    dev = torch.device("cuda:0")
    x, v, p = workloads.state(w)
    d, t = workloads.quadratic_vectors(w)
    dx, dv = torch.from_numpy(x).to(dev), torch.from_numpy(v).to(dev)
    dp = dx.clone()
    dd, dt = torch.from_numpy(d).to(dev), torch.from_numpy(t).to(dev)
    gpu = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                        seed=w.seed, flags=PSOPS_QUADRATIC)
    gpu.set_quadratic(dd, dt)
    gpu.eval_quadratic()
    ref = oracle.RefSwarm(x[:, :w.N], v[:, :w.N], p[:, :w.N], m_max=w.omega, m_min=w.omega, t_max=1,
                          c1=w.c1, c2=w.c2, seed=w.seed, nthreads=NTHREADS)
    del x, v, p
    loss = oracle.quadratic_losses(ref.x, d, t, nthreads=NTHREADS)
    for s in range(syncs):
        assert np.array_equal(gpu.losses().view(np.uint32), loss.view(np.uint32)), s
        gpu.sync(0, w.lam)
        ref.sync(loss, 0, w.lam)
        g, improved, pl = gpu.info()
        assert g == ref.g and np.array_equal(improved, ref.improved), s
        assert np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32)), s
        loss = oracle.quadratic_losses(ref.x, d, t, nthreads=NTHREADS)
        if s in (0, 19, 99) or s == syncs - 1:
            for name, tdev, want in (("x", dx, ref.x), ("v", dv, ref.v), ("pbest", dp, ref.p)):
                assert gpu_util.device_compare(tdev[:, :w.N], want, f"cfg5 s={s} {name}") == 0
    assert np.array_equal(gpu.losses().view(np.uint32), loss.view(np.uint32))
    gpu.close()


# ---------------------------------------------------------------------------
# Parameter averaging.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("K,N,ld,offset", [(1, 100, 100, 0), (2, 1001, 1004, 0), (16, 300_002, 300_004, 0),
                                           (7, 999, 999, 1), (32, 70_000, 70_000, 0), (33, 5, 8, 0)])
def test_average_bit_exact(K, N, ld, offset):
    x, v, p = _swarm(K, N, K + N)
    pair = Pair(x, v, p, N, ld=ld, offset=offset, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    pair.gpu.average()
    pair.ref.average()
    got = pair.dx.host()
    assert np.array_equal(got.view(np.uint32), pair.ref.x.view(np.uint32))
    assert np.array_equal(pair.dv.host(), v) and np.array_equal(pair.dp.host(), p)   # untouched
    pair.check_canaries()
    # averaging then a sync still follows the oracle
    pair.sync(np.linspace(1, 2, K).astype(np.float32))
    pair.check_selection()
    pair.check_state("after average")
    pair.close()


# ---------------------------------------------------------------------------
# Host-buffer entry point, row access, determinism, resume.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("pinned", [False, True])
def test_sync_host_matches_oracle(pinned):
    w = workloads.CONFIGS["cfg2"].scaled(N=2_500_001, S=3)     # several pipeline ranges + ragged tail
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    pair = Pair(x, v, p, w.N, ld=w.ld, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)
    h_in = torch.from_numpy(x.copy())
    h_out = torch.full((w.K, w.ld), 123.0)
    if pinned:
        h_in, h_out = h_in.pin_memory(), h_out.pin_memory()
    for s in range(w.S):
        # the workers' weights arrive from the host each time
        h_in[:, :w.N] = torch.from_numpy(pair.ref.x)
        pair.gpu.sync_host(h_in, table[s], 0, w.lam, h_out)
        pair.ref.sync(table[s], 0, w.lam)
        pair.check_selection()
        assert assert_close(h_out.numpy()[:, :w.N], pair.ref.x, "host out") == 0
        assert torch.all(h_out[:, w.N:] == 123.0)
        pair.check_state(f"sync_host s={s}")
    pair.check_canaries()
    pair.close()


def test_get_and_set_weights_rows():
    K, N = 3, 1001
    x, v, p = _swarm(K, N, 1)
    pair = Pair(x, v, p, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    for which, src in ((PSOPS_X, x), (PSOPS_V, v), (PSOPS_PBEST, p)):
        for k in range(K):
            assert np.array_equal(pair.gpu.row(which, k), src[k])
    new = np.arange(N, dtype=np.float32)
    binding.psops_set_weights(pair.gpu.ctx, PSOPS_V, 1, new)
    assert np.array_equal(pair.gpu.row(PSOPS_V, 1), new)
    dev_dst = torch.empty(N, device="cuda")
    binding.psops_get_weights(pair.gpu.ctx, PSOPS_X, 2, dev_dst)
    assert np.array_equal(dev_dst.cpu().numpy(), x[2])
    with pytest.raises(binding.PsopsError) as e:
        pair.gpu.row(PSOPS_GBEST)
    assert e.value.code == binding.PSOPS_ESTATE
    with pytest.raises(binding.PsopsError):
        pair.gpu.row(PSOPS_X, K)
    pair.check_canaries()
    pair.close()


def test_deterministic_and_resumable():
    w = workloads.CONFIGS["cfg1"].scaled(N=50_001, S=10)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    kw = dict(N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)

    def fresh():
        return [torch.from_numpy(a).cuda() for a in (x, v, p)]

    a = fresh()
    sa = binding.Swarm(*a, **kw)
    for s in range(10):
        sa.set_losses(table[s])
        sa.sync()
    b = fresh()
    sb = binding.Swarm(*b, **kw)
    for s in range(5):
        sb.set_losses(table[s])
        sb.sync()
    step, pl = sb.state()
    assert step == 5
    sb.close()
    sc = binding.Swarm(*b, **kw)          # new context on the same tensors
    sc.set_state(step, pl)
    for s in range(5, 10):
        sc.set_losses(table[s])
        sc.sync()
    torch.cuda.synchronize()
    for ta, tb in zip(a, b):
        assert torch.equal(ta, tb)
    assert sa.info()[0] == sc.info()[0] and np.array_equal(sa.info()[2], sc.info()[2])
    sa.close()
    sc.close()


@pytest.mark.parametrize("K", [4, 7, 16, 40])          # single launch (two depths), selecting snapshot + row-split
def test_sync_recorded_in_a_cuda_graph_replays_with_a_running_step_counter(K):   # update, selection + snapshot + update
    w = workloads.CONFIGS["cfg1"].scaled(N=40_001, S=8).with_particles(K)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        t = [torch.from_numpy(a).cuda() for a in (x, v, p)]
        lbuf = torch.zeros(w.K, device="cuda")
    stream.synchronize()
    sw = binding.Swarm(*t, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed,
                       stream=stream.cuda_stream)
    ref = oracle.RefSwarm(x[:, :w.N], v[:, :w.N], p[:, :w.N], m_max=w.omega, m_min=w.omega, t_max=1,
                          c1=w.c1, c2=w.c2, seed=w.seed)
    # one eager sync first (also warms the launch path), then record one sync
    with torch.cuda.stream(stream):
        lbuf.copy_(torch.from_numpy(table[0]))
        sw.set_losses(lbuf)
        sw.sync()
    ref.sync(table[0])
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        sw.set_losses(lbuf)
        sw.sync()
    # capture only records: the state must be unchanged
    assert assert_close(t[0].cpu().numpy()[:, :w.N], ref.x, "after capture") == 0
    for s in range(1, w.S):
        with torch.cuda.stream(stream):
            lbuf.copy_(torch.from_numpy(table[s]))
            graph.replay()
        ref.sync(table[s])
        stream.synchronize()
        g, improved, pl = sw.info()
        assert g == ref.g and np.array_equal(improved, ref.improved)
        assert np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32))
    for got, want, name in ((t[0], ref.x, "x"), (t[1], ref.v, "v"), (t[2], ref.p, "pbest")):
        assert assert_close(got.cpu().numpy()[:, :w.N], want, name) == 0
    assert sw.state()[0] == w.S                     # the device-side counter saw every replay
    sw.close()


def test_runs_on_a_side_stream_and_counts_launches():
    K, N = 4, 20_000
    x, v, p = _swarm(K, N, 4)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        t = [torch.from_numpy(a).cuda() for a in (x, v, p)]
    stream.synchronize()
    sw = binding.Swarm(*t, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=8, stream=stream.cuda_stream)
    ref = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=8)
    loss = np.array([4, 3, 2, 1], np.float32)
    sw.set_losses(loss)
    sw.sync()
    ref.sync(loss)
    stream.synchronize()
    assert sw.launches == 1                        # four particles: selection and update are one launch
    assert assert_close(t[0].cpu().numpy(), ref.x) == 0
    sw.average()
    assert sw.launches == 2
    sw.close()
    sw = binding.Swarm(*t, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=8, stream=stream.cuda_stream,
                       flags=PSOPS_SEPARATE_SELECT)
    sw.set_losses(loss)
    sw.sync()
    assert sw.launches == 2                        # selection kernel + update kernel
    sw.close()


def test_device_errors_and_call_order():
    K, N = 2, 64
    x, v, p = _swarm(K, N, 4)
    t = [torch.from_numpy(a).cuda() for a in (x, v, p)]
    sw = binding.Swarm(*t, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=8)
    before = [a.clone() for a in t]
    codes = []
    for fn in (lambda: sw.sync(),                                   # no losses yet
               lambda: sw.set_losses(np.array([np.nan, 1.0], np.float32)),
               lambda: sw.info(),
               lambda: sw.eval_quadratic(),
               lambda: sw.set_quadratic(t[0], t[1])):               # no QUADRATIC workspace
        with pytest.raises(binding.PsopsError) as e:
            fn()
        codes.append(e.value.code)
    assert codes == [binding.PSOPS_ESTATE, binding.PSOPS_ENAN, binding.PSOPS_ESTATE,
                     binding.PSOPS_ESTATE, binding.PSOPS_EWORKSPACE]
    sw.set_losses([1.0, 2.0])
    for bad in (lambda: sw.sync(-1, 1.0), lambda: sw.sync(0, 0.5), lambda: sw.sync(0, float("nan")),
                lambda: sw.sync(0, float("inf"))):
        with pytest.raises(binding.PsopsError) as e:
            bad()
        assert e.value.code == binding.PSOPS_EINVAL
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(t, before))        # nothing was touched
    assert sw.launches == 0
    # misaligned or undersized workspace
    cfg = sw.cfg
    ws = torch.empty(binding.psops_workspace_bytes(cfg) + 512, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.PsopsError) as e:
        binding.psops_create(cfg, *t, ws[4:], ws.numel() - 4)
    assert e.value.code == binding.PSOPS_EWORKSPACE
    with pytest.raises(binding.PsopsError) as e:
        binding.psops_create(cfg, *t, ws, 16)
    assert e.value.code == binding.PSOPS_EWORKSPACE
    sw.close()


def test_element_indices_beyond_32_bits():
    """N just above 2^32 (the Philox counter word d >> 1 passes 2^31, element
    offsets need 64 bits, ragged last quad).  The state is drawn on the device
    by torch's seeded generator; the oracle follows columns sampled around the
    interesting boundaries, read back before the first sync."""
    gpu_util.ensure_library()
    K, N = 2, (1 << 32) + 4099
    ld = (N + 1023) // 1024 * 1024
    free, _ = torch.cuda.mem_get_info()
    if free < 3 * K * ld * 4 + (8 << 30):
        pytest.skip("needs about 110 GB of free device memory")
    gen = torch.Generator(device="cuda").manual_seed(2033)
    dx = torch.empty((K, ld), dtype=torch.float32, device="cuda").normal_(0.0, 0.01, generator=gen)
    dv = torch.empty((K, ld), dtype=torch.float32, device="cuda").normal_(0.0, 1e-3, generator=gen)
    dp = dx.clone()
    edges = [0, 1 << 31, (1 << 32) - 4, 1 << 32, N - 8]
    cols = np.unique(np.concatenate(
        [np.arange(max(0, e - 6), min(N, e + 10)) for e in edges]
        + [np.random.default_rng(1).integers(0, N, size=500)]).astype(np.int64))
    dcols = torch.from_numpy(cols).cuda()
    xs, vs = dx[:, dcols].cpu().numpy(), dv[:, dcols].cpu().numpy()
    pad_before = [t[:, N:].clone() for t in (dx, dv, dp)]
    sw = binding.Swarm(dx, dv, dp, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=0xABCDEF0123456789)
    ref = oracle.RefSwarm(xs, vs, xs, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5,
                          seed=0xABCDEF0123456789, elem_index=cols)
    for loss in ([0.9, 0.4], [0.3, 0.6], [0.35, 0.1]):
        sw.set_losses(np.array(loss, np.float32))
        sw.sync()
        ref.sync(np.array(loss, np.float32))
        g, improved, _ = sw.info()
        assert g == ref.g and np.array_equal(improved, ref.improved)
    for name, t, want in (("x", dx, ref.x), ("v", dv, ref.v), ("pbest", dp, ref.p)):
        assert assert_close(t[:, dcols].cpu().numpy(), want, name) == 0
    for t, before in zip((dx, dv, dp), pad_before):
        assert torch.equal(t[:, N:], before)               # padding untouched
    sw.close()


def test_sync_host_in_place_with_history_schedule_and_kept_gbest():
    """Host-buffer sync where the output overwrites the input, Eq. 5 and lambda
    vary per call, and gBest comes from the history (so some pipeline ranges
    read the remembered row and others row g)."""
    w = workloads.CONFIGS["cfg6"].scaled(N=1_300_003, S=6)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    table[3] = table[3] + np.float32(3.0)           # worse than anything before: history must hold
    gpu_util.ensure_library()
    dx, dv, dp = (gpu_util.DeviceRows(a, w.N, w.ld) for a in (x, v, p))
    sw = binding.Swarm(dx.rows, dv.rows, dp.rows, N=w.N, m_max=w.m_max, m_min=w.m_lo, t_max=w.t_max,
                       c1=w.c1, c2=w.c2, seed=w.seed, flags=binding.PSOPS_GBEST_HISTORY)
    ref = oracle.RefSwarm(x[:, :w.N], v[:, :w.N], p[:, :w.N], m_max=w.m_max, m_min=w.m_lo, t_max=w.t_max,
                          c1=w.c1, c2=w.c2, seed=w.seed, nthreads=NTHREADS, history=True)
    h = torch.from_numpy(x.copy()).pin_memory()
    for s in range(w.S):
        t, lam = w.schedule(s * 97)                  # spread over the epochs
        sw.sync_host(h, table[s], t, lam)            # in place
        ref.sync(table[s], t, lam, want_gbest=True)
        g, improved, pl = sw.info()
        assert g == ref.g and np.array_equal(improved, ref.improved)
        assert assert_close(h.numpy()[:, :w.N], ref.x, f"in-place host s={s}") == 0
        assert np.array_equal(sw.row(PSOPS_GBEST), ref.gbest)
    assert not np.array_equal(ref.gbest, ref.x[ref.g])          # the remembered row was in use
    for d, want in ((dx, ref.x), (dv, ref.v), (dp, ref.p)):
        assert assert_close(d.host(), want, "device state") == 0
        d.check_canaries("sync_host history")
    sw.close()


def test_sync_host_with_fused_fitness():
    w = workloads.CONFIGS["cfg5"].scaled(N=2_600_005, S=3)
    pair, d, t = _quadratic_pair(w)
    pair.gpu.eval_quadratic()
    loss = oracle.quadratic_losses(pair.ref.x, d, t, nthreads=NTHREADS)
    h_in = torch.from_numpy(workloads.state(w)[0]).pin_memory()
    h_out = torch.zeros_like(h_in).pin_memory()
    for s in range(w.S):
        h_in[:, :w.N] = torch.from_numpy(pair.ref.x)
        pair.gpu.sync_host(h_in, loss, 0, w.lam, h_out)
        pair.ref.sync(loss, 0, w.lam)
        pair.check_selection()
        loss = oracle.quadratic_losses(pair.ref.x, d, t, nthreads=NTHREADS)
        assert np.array_equal(pair.gpu.losses().view(np.uint32), loss.view(np.uint32))
        assert assert_close(h_out.numpy()[:, :w.N], pair.ref.x, "host out") == 0
    pair.check_state("sync_host fused fitness")
    pair.check_canaries()
    pair.close()


def test_two_contexts_on_two_streams_do_not_interfere():
    w = workloads.CONFIGS["cfg2"].scaled(N=400_001, S=6)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    pairs, streams = [], [torch.cuda.Stream(), torch.cuda.Stream()]
    refs = []
    for i, st in enumerate(streams):
        with torch.cuda.stream(st):
            t = [torch.from_numpy(a).cuda() for a in (x, v, p)]
        st.synchronize()
        pairs.append((t, binding.Swarm(*t, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                                       seed=w.seed + i, stream=st.cuda_stream)))
        refs.append(oracle.RefSwarm(x[:, :w.N], v[:, :w.N], p[:, :w.N], m_max=w.omega, m_min=w.omega,
                                    t_max=1, c1=w.c1, c2=w.c2, seed=w.seed + i, nthreads=NTHREADS))
    dt = torch.from_numpy(table).cuda()
    torch.cuda.synchronize()
    for s in range(w.S):                             # enqueue both without waiting in between
        for i, (t, sw) in enumerate(pairs):
            sw.set_losses(dt[(s + i) % w.S])
            sw.sync()
    torch.cuda.synchronize()
    for i, ref in enumerate(refs):
        for s in range(w.S):
            ref.sync(table[(s + i) % w.S])
        for got, want in zip(pairs[i][0], (ref.x, ref.v, ref.p)):
            assert assert_close(got.cpu().numpy()[:, :w.N], want, f"context {i}") == 0
        pairs[i][1].close()


def test_ssgd_of_one_local_step_equals_averaging_on_device():
    """Section II-B: with a sync every iteration, averaging the workers' weights
    after one local step w + alpha g_k is the SSGD update (up to rounding)."""
    K, N = 8, 200_003
    rng = np.random.default_rng(3)
    w0 = np.tile(rng.standard_normal(N).astype(np.float32), (K, 1))
    g = rng.standard_normal((K, N)).astype(np.float32)
    alpha = np.float32(-0.125)
    zeros = np.zeros_like(w0)
    a = Pair((w0 + alpha * g).astype(np.float32), zeros, zeros, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    b = Pair(w0, zeros, zeros, N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    a.gpu.average()
    dg = gpu_util.DeviceRows(g, N, (N + 3) // 4 * 4)
    b.gpu.ssgd(dg.rows, float(alpha))
    pa, ss = a.dx.host(), b.dx.host()
    scale = np.abs(w0[0]) + np.abs(alpha) * np.abs(g).max(axis=0)
    assert np.all(np.abs(pa - ss) <= 16 * 2.0 ** -24 * scale)
    a.close()
    b.close()


def test_subnormal_overflow_and_nan_values_follow_ieee_on_both_sides():
    """No flush-to-zero anywhere: subnormal weights and velocities stay
    subnormal; overflow gives inf and inf - inf gives NaN in the same elements
    on the GPU and in the oracle."""
    K, N = 4, 4099
    rng = np.random.default_rng(77)
    x = (rng.standard_normal((K, N)) * 1e-39).astype(np.float32)            # subnormal
    v = (rng.standard_normal((K, N)) * 3e-42).astype(np.float32)
    p = (rng.standard_normal((K, N)) * 1e-38).astype(np.float32)
    x[:, 100:200] = (rng.uniform(-1, 1, (K, 100)) * 3e38).astype(np.float32)   # overflows in Eq. 6/7
    v[:, 100:200] = (rng.uniform(-1, 1, (K, 100)) * 3e38).astype(np.float32)
    x[1, 300] = np.inf
    x[2, 301] = -np.inf
    p[3, 302] = np.nan
    assert np.any((np.abs(x) > 0) & (np.abs(x) < 1.17e-38))
    pair = Pair(x, v, p, N, m_max=0.9, m_min=0.9, c1=2.0, c2=2.0, seed=5)
    with np.errstate(all="ignore"):
        for s, loss in enumerate(([4, 3, 2, 1], [1, 2, 3, 4], [2, 1, 2, 1])):
            pair.sync(np.array(loss, np.float32))
            pair.check_selection()
            for d, want, name in ((pair.dx, pair.ref.x, "x"), (pair.dv, pair.ref.v, "v"), (pair.dp, pair.ref.p, "p")):
                got = d.host()
                assert np.array_equal(np.isnan(got), np.isnan(want)), name
                ok = ~np.isnan(want)
                assert np.array_equal(got[ok], want[ok]), f"{name} s={s}"      # values (+0 == -0)
    sub = (np.abs(pair.ref.v) > 0) & (np.abs(pair.ref.v) < 1.17e-38)
    assert sub.any() and np.isinf(pair.ref.x).any() and np.isnan(pair.ref.x).any()
    pair.close()


def test_host_register_pins_a_numpy_buffer_for_sync_host():
    w = workloads.CONFIGS["cfg2"].scaled(N=1_500_003, S=2)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    pair = Pair(x, v, p, w.N, ld=w.ld, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2, seed=w.seed)
    h = x.copy()                                        # plain numpy memory
    binding.psops_host_register(h)
    binding.psops_host_register(h)                      # twice is fine
    assert torch.from_numpy(h).is_pinned()
    try:
        for s in range(w.S):
            pair.gpu.sync_host(h, table[s], 0, w.lam)   # in place
            pair.ref.sync(table[s], 0, w.lam)
            assert assert_close(h[:, :w.N], pair.ref.x, "registered host buffer") == 0
    finally:
        binding.psops_host_unregister(h)
    with pytest.raises(binding.PsopsError):
        binding.psops_host_unregister(h)                # no longer registered
    pair.close()
