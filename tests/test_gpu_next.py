"""GPU parity of the widened rows: the Table II schedule, gBest from history,
the particle-sharded sync (shards emulated one after another on one GPU -- no
kernel waits on another) and the SSGD baseline."""
import numpy as np
import pytest
import torch

import oracle
from paper_2009_03816_b200 import binding, sharded, workloads
from paper_2009_03816_b200.binding import PSOPS_GBEST, PSOPS_GBEST_HISTORY, PSOPS_X

import gpu_util
from gpu_util import NTHREADS, Pair, assert_close

pytestmark = pytest.mark.gpu


def _swarm(K, N, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((K, N)).astype(np.float32)
    v = (0.1 * rng.standard_normal((K, N))).astype(np.float32)
    p = (x + 0.5 * rng.standard_normal((K, N))).astype(np.float32)
    return x, v, p


def test_table2_schedule_every_sync():
    """m from Eq. 5 falling 0.9 -> 0.3 over t_max iterations, c1 = 0.2,
    c2 = 0.9, lambda = epoch index 1..25 (Table II), 585 syncs."""
    w = workloads.CONFIGS["cfg6"]
    assert w.t_max == 5850 and w.schedule(0) == (10, 1.0) and w.schedule(584) == (5850, 25.0)
    x, v, p = workloads.state(w)
    table = workloads.losses(w)
    pair = Pair(x, v, p, w.N, ld=w.ld, m_max=w.m_max, m_min=w.m_lo, t_max=w.t_max, c1=w.c1, c2=w.c2,
                seed=w.seed)
    for s in range(w.S):
        t, lam = w.schedule(s)
        pair.sync(table[s], t, lam)
        pair.check_selection()
        if s % 45 == 0 or s == w.S - 1:
            pair.check_state(f"cfg6 s={s}")
    assert pair.inexact == 0
    pair.check_canaries()
    pair.close()


@pytest.mark.parametrize("N,ld,offset", [(10_007, None, 0), (1001, 1001, 1)])
def test_history_gbest_matches_oracle(N, ld, offset):
    K = 6
    x, v, p = _swarm(K, N, 31)
    ld = (N + 3) // 4 * 4 if ld is None else ld
    gpu_util.ensure_library()
    dx, dv, dp = (gpu_util.DeviceRows(a, N, ld, offset) for a in (x, v, p))
    sw = binding.Swarm(dx.rows, dv.rows, dp.rows, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=9,
                       flags=PSOPS_GBEST_HISTORY)
    ref = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=9, history=True)
    with pytest.raises(binding.PsopsError):
        sw.row(PSOPS_GBEST)                              # nothing remembered yet
    rng = np.random.default_rng(3)
    kept = 0
    for s in range(12):
        loss = rng.random(K).astype(np.float32) + np.float32(0.3 * (s % 3))   # often worse than before
        if s == 7:
            loss[2] = ref.history["loss"][0]             # equal to the remembered loss: not better
        sw.set_losses(loss)
        sw.sync()
        before = ref.history["loss"][0]
        ref.sync(loss, want_gbest=True)
        kept += int(ref.history["loss"][0] == before)
        g, improved, pl = sw.info()
        assert g == ref.g and np.array_equal(improved, ref.improved)
        hl, valid = sw.history()
        assert valid and np.float32(hl) == ref.history["loss"][0]
        assert np.array_equal(sw.row(PSOPS_GBEST), ref.gbest)
        for d, want, name in ((dx, ref.x, "x"), (dv, ref.v, "v"), (dp, ref.p, "pbest")):
            assert assert_close(d.host(), want, f"history s={s} {name}") == 0
    assert kept >= 4                                     # the remembered row really was reused
    for d in (dx, dv, dp):
        d.check_canaries("history")
    # resume: the remembered row and loss move to a new context
    hl, _ = sw.history()
    row = sw.row(PSOPS_GBEST)
    step, pl = sw.state()
    sw.close()
    sw2 = binding.Swarm(dx.rows, dv.rows, dp.rows, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=9,
                        flags=PSOPS_GBEST_HISTORY)
    sw2.set_state(step, pl)
    binding.psops_set_history(sw2.ctx, hl, row)
    loss = np.full(K, 5.0, np.float32)
    sw2.set_losses(loss)
    sw2.sync()
    ref.sync(loss)
    assert assert_close(dx.host(), ref.x, "after resume") == 0
    sw2.close()


@pytest.mark.parametrize("counts", [[1, 1, 1, 1], [2, 2, 2, 2], [3, 1, 4], [8], [30, 10, 30], [33, 37]])
def test_particle_shards_reproduce_the_unsharded_sync(counts):
    """Every shard is a context of its own with its own rows; they are driven
    one after another through the calls a multi-GPU run makes.  The result
    must be that of one unsharded swarm (the oracle)."""
    K = sum(counts)
    N = 20_003 if K <= 8 else 3_001          # shards whose improved bits straddle 32-bit words
    ld = (N + 3) // 4 * 4
    x, v, p = _swarm(K, N, 5)
    gpu_util.ensure_library()
    ref = oracle.RefSwarm(x, v, p, m_max=0.9, m_min=0.3, t_max=40, c1=0.2, c2=0.9, seed=77, nthreads=NTHREADS)
    shards, first = [], 0
    for n in counts:
        rows = [gpu_util.DeviceRows(a[first:first + n], N, ld) for a in (x, v, p)]
        sw = binding.Swarm(rows[0].rows, rows[1].rows, rows[2].rows, N=N, m_max=0.9, m_min=0.3, t_max=40,
                           c1=0.2, c2=0.9, seed=77, k_first=first, K_total=K)
        shards.append((first, n, rows, sw))
        first += n
    gbest = torch.zeros(N, device="cuda")
    rng = np.random.default_rng(8)
    for s in range(6):
        loss = rng.random(K).astype(np.float32)
        if s == 3:
            loss[K - 1] = loss.min()                     # tie: lowest index wins on every shard
        dl = torch.from_numpy(loss).cuda()
        gs = []
        for _, _, _, sw in shards:
            sw.set_losses(dl)
            gs.append(sw.shard_select())
        assert len(set(gs)) == 1
        owner, row = sharded.owner_of(gs[0], counts)
        binding.psops_get_weights(shards[owner][3].ctx, PSOPS_X, row, gbest)
        for _, _, _, sw in shards:
            sw.shard_update(gbest, 4 * s, 1.0 + s)
        ref.sync(loss, 4 * s, 1.0 + s, want_gbest=True)
        assert gs[0] == ref.g
        assert np.array_equal(gbest.cpu().numpy(), ref.gbest)
        for f, n, rows, sw in shards:
            g, improved, pl = sw.info()
            assert np.array_equal(improved, ref.improved) and np.array_equal(pl, ref.pbest_loss)
            for d, want, name in zip(rows, (ref.x, ref.v, ref.p), "xvp"):
                assert assert_close(d.host(), want[f:f + n], f"shard@{f} s={s} {name}") == 0
    for _, _, rows, sw in shards:
        for d in rows:
            d.check_canaries("shard")
        if len(counts) > 1:
            with pytest.raises(binding.PsopsError) as e:
                sw.sync()                                # a shard cannot sync on its own
            assert e.value.code == binding.PSOPS_ESTATE
        with pytest.raises(binding.PsopsError) as e:
            sw.shard_update(gbest)                       # update without a selection
        assert e.value.code == binding.PSOPS_ESTATE
        sw.close()


def test_shards_update_in_ranges_owner_reads_its_own_row_and_gbest_is_kept():
    """The multi-GPU driver's calls, shard after shard on one GPU: the update
    goes over the element ranges of a chunked broadcast; the shard that holds
    gBest reads the row in place from its own weights; with PSOPS_KEEP_GBEST
    every shard keeps a copy of the row it was given."""
    counts = [3, 1, 4]
    K, N = sum(counts), 50_003
    ld = (N + 1023) // 1024 * 1024
    x, v, p = _swarm(K, N, 12)
    gpu_util.ensure_library()
    ref = oracle.RefSwarm(x, v, p, m_max=0.9, m_min=0.3, t_max=40, c1=0.2, c2=0.9, seed=5, nthreads=NTHREADS)
    shards, first = [], 0
    for n in counts:
        rows = [gpu_util.DeviceRows(a[first:first + n], N, ld) for a in (x, v, p)]
        sw = binding.Swarm(rows[0].rows, rows[1].rows, rows[2].rows, N=N, m_max=0.9, m_min=0.3, t_max=40,
                           c1=0.2, c2=0.9, seed=5, k_first=first, K_total=K, flags=binding.PSOPS_KEEP_GBEST)
        shards.append((first, n, rows, sw))
        first += n
    bounds = sharded.range_bounds(N, 4)
    assert len(bounds) == 4 and bounds[-1][1] == N and N % 4 == 3
    received = torch.zeros(N, device="cuda")           # what a broadcast would deliver to the other shards
    rng = np.random.default_rng(2)
    for s in range(5):
        loss = rng.random(K).astype(np.float32)
        loss[[2, 3, 6, 0, 5][s]] = 0.0                 # gBest on every shard in turn, first and last rows too
        dl = torch.from_numpy(loss).cuda()
        gs = [sw.set_losses(dl) or sw.shard_select() for _, _, _, sw in shards]
        assert len(set(gs)) == 1
        owner, row = sharded.owner_of(gs[0], counts)
        received.copy_(shards[owner][3].x[row, :N])    # leaves the owner before anything is overwritten
        for r, (_, _, _, sw) in enumerate(shards):
            src = sw.x[row, :N] if r == owner else received
            for a, b in bounds:
                sw.shard_update_range(src, a, b, 4 * s, 1.0 + s)
        ref.sync(loss, 4 * s, 1.0 + s, want_gbest=True)
        assert gs[0] == ref.g
        for f, n, rows, sw in shards:
            g, improved, pl = sw.info()
            assert np.array_equal(improved, ref.improved) and np.array_equal(pl, ref.pbest_loss)
            assert np.array_equal(sw.row(PSOPS_GBEST), ref.gbest)
            for d, want, name in zip(rows, (ref.x, ref.v, ref.p), "xvp"):
                assert assert_close(d.host(), want[f:f + n], f"shard@{f} s={s} {name}") == 0
    _, _, rows, sw = shards[0]
    # ranges must come left to right, on quad boundaries, after a selection
    sw.set_losses(dl)
    sw.shard_select()
    with pytest.raises(binding.PsopsError) as e:
        sw.shard_select()                                # a selection whose update is still due
    assert e.value.code == binding.PSOPS_ESTATE
    for a, b, code in ((4, 8, binding.PSOPS_ESTATE), (0, 6, binding.PSOPS_EINVAL), (0, N + 1, binding.PSOPS_EINVAL)):
        with pytest.raises(binding.PsopsError) as e:
            sw.shard_update_range(received, a, b)
        assert e.value.code == code
    sw.shard_update_range(received, 0, 1024)
    with pytest.raises(binding.PsopsError) as e:
        sw.shard_select()                                # an update is half done
    assert e.value.code == binding.PSOPS_ESTATE
    with pytest.raises(binding.PsopsError) as e:
        sw.shard_update_range(received, 0, 1024)         # the same range again
    assert e.value.code == binding.PSOPS_ESTATE
    sw.shard_update_range(received, 1024, N)
    # the whole-swarm operations are refused on a shard
    for fn in (sw.average, lambda: sw.ssgd(rows[0].rows, -0.1)):
        with pytest.raises(binding.PsopsError) as e:
            fn()
        assert e.value.code == binding.PSOPS_ESTATE
    for _, _, rows, sw in shards:
        for d in rows:
            d.check_canaries("shard ranges")
        sw.close()


def test_sharded_driver_single_rank():
    """The driver class on one rank (no process group): same calls, same result."""
    K, N = 4, 5000
    x, v, p = _swarm(K, N, 6)
    t = [torch.from_numpy(a).cuda() for a in (x, v, p)]
    sw = binding.Swarm(*t, N=N, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1, k_first=0, K_total=K)
    drv = sharded.ShardedSync(sharded.swarm_engine(sw), [K], N, torch.device("cuda"))
    ref = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=1)
    for s in range(3):
        loss = np.array([3, 1, 2, 4], np.float32) + s
        g = drv.sync(torch.from_numpy(loss).cuda())
        ref.sync(loss)
        assert g == ref.g
    assert assert_close(t[0].cpu().numpy(), ref.x, "driver x") == 0
    sw.close()


@pytest.mark.parametrize("K,N,ld,gld,offset", [(1, 100, 100, 100, 0), (4, 10_001, 10_004, 10_008, 0),
                                               (7, 999, 999, 1001, 1), (16, 300_002, 300_032, 300_032, 0)])
def test_ssgd_bit_exact(K, N, ld, gld, offset):
    rng = np.random.default_rng(K + N)
    x = np.tile(rng.standard_normal(N).astype(np.float32), (K, 1))
    g = rng.standard_normal((K, N)).astype(np.float32)
    _, v, p = _swarm(K, N, 2)
    pair = Pair(x, v, p, N, ld=ld, offset=offset, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    dg = gpu_util.DeviceRows(g, N, gld, offset)
    pair.gpu.ssgd(dg.rows, -0.05)
    oracle.ssgd(pair.ref.x, g, -0.05)
    got = pair.dx.host()
    assert np.array_equal(got.view(np.uint32), pair.ref.x.view(np.uint32))
    assert np.array_equal(pair.dv.host(), v) and np.array_equal(pair.dp.host(), p)
    assert np.array_equal(dg.host(), g)
    pair.check_canaries("ssgd")
    dg.check_canaries("ssgd grad")
    pair.close()
