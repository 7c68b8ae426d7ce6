"""The N>1 plumbing (independent replicas: barrier, max-over-ranks timing, summed
units) exercised as two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

from conftest import ROOT

WORKER = textwrap.dedent("""
    import json, os, sys, time
    sys.path.insert(0, os.environ["PSOPS_ROOT"])
    from paper_2009_03816_b200 import replicas
    r = replicas.init_from_env(backend="gloo")
    assert r.world == 2 and r.backend == "gloo"
    replicas.barrier(r)
    mine = 1.0 + r.rank                       # rank 1 is the slow one
    units = 100.0 * (r.rank + 1)
    rate, slowest = replicas.whole_job_rate(r, units, mine)
    mx = replicas.max_over_ranks(r, float(r.rank))
    sm = replicas.sum_over_ranks(r, 1.0)
    replicas.barrier(r)
    if r.is_root:
        print(json.dumps({"rate": rate, "slowest": slowest, "max": mx, "sum": sm}))
    replicas.finish(r)
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_aggregate_like_the_benchmark(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PSOPS_ROOT=ROOT,
                   CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    import json
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert res["slowest"] == 2.0 and res["max"] == 1.0 and res["sum"] == 2.0
    assert res["rate"] == 300.0 / 2.0                     # all ranks' units / slowest rank's time
    assert outs[1][0].strip() == ""                        # only rank 0 prints


def test_single_process_needs_no_group():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    code = ("import sys; sys.path.insert(0, %r); from paper_2009_03816_b200 import replicas; "
            "r = replicas.init_from_env(); assert r.world == 1 and r.is_root; "
            "assert replicas.whole_job_rate(r, 10.0, 2.0) == (5.0, 2.0); replicas.barrier(r)" % ROOT)
    subprocess.run([sys.executable, "-c", code], env=env, check=True, timeout=120)


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


# ---------------------------------------------------------------------------
# Particle-sharded sync: collective ordering and ownership, two gloo ranks.
# The engine behind the driver is the CPU oracle run on the full swarm by every
# rank (tests may use the oracle); what is checked is the exchange itself.
# ---------------------------------------------------------------------------
SHARD_WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, os.environ["PSOPS_ROOT"])
    import numpy as np, torch
    import torch.distributed as dist
    import oracle
    from paper_2009_03816_b200 import replicas, sharded
    r = replicas.init_from_env(backend="gloo")
    counts = [3, 2]
    K, N = 5, 257
    rng = np.random.default_rng(0)
    x = rng.standard_normal((K, N)).astype(np.float32); v = np.zeros_like(x); p = x.copy()
    full = oracle.RefSwarm(x, v, p, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=4)
    first = sharded.first_index(r.rank, counts)

    class Engine:                       # holds only this rank's rows of the reference swarm
        def __init__(self): self.log = []
        def set_losses(self, all_losses): self.losses = all_losses.numpy().copy()
        def shard_select(self):
            self.g = oracle.argmin(self.losses); self.pre = full.x.copy(); return self.g
        def row(self, row):             # the owner sends this memory itself, nothing is copied out
            self.log.append(("row", row)); return torch.from_numpy(full.x[first + row])
        def shard_update_range(self, gbest, a, b, t, lam):
            self.log.append(("range", a, b))
            assert np.array_equal(gbest.numpy()[a:b], self.pre[self.g][a:b]), "range has not arrived"
            if b == N:                  # last range: the whole row is here; now the weights may change
                assert np.array_equal(gbest.numpy(), self.pre[self.g]), "broadcast row is not gBest"
                full.sync(self.losses, t, lam, want_gbest=True)
                assert np.array_equal(full.gbest, self.pre[self.g])

    eng = Engine()
    drv = sharded.ShardedSync(eng, counts, N, torch.device("cpu"), pieces=3, quantum=4)
    assert drv.bounds == [(0, 88), (88, 176), (176, 257)]
    gs = []
    table = np.array([[5, 4, 3, 2, 1], [1, 2, 3, 4, 5], [2, 2, 1, 1, 3]], np.float32)
    for s in range(3):
        mine = torch.from_numpy(table[s, first:first + counts[r.rank]].copy())
        gs.append(drv.sync(mine))
        assert np.array_equal(eng.losses, table[s]), "all-gather order"
    # equal shards take the single-collective gather: same losses in the same order
    class Probe(Engine):
        def shard_update_range(self, gbest, a, b, t, lam): pass
    probe = Probe()
    drv2 = sharded.ShardedSync(probe, [2, 2], N, torch.device("cpu"), pieces=1)
    drv2.sync(torch.tensor([10.0 + r.rank, 20.0 + r.rank]))
    assert probe.losses.tolist() == [10.0, 20.0, 11.0, 21.0], probe.losses
    print(json.dumps({"rank": r.rank, "g": gs, "log": eng.log}))
    replicas.finish(r)
""")


def test_sharded_exchange_two_gloo_ranks(tmp_path):
    import json
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PSOPS_ROOT=ROOT,
                   CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err
    res = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    assert res[0]["g"] == res[1]["g"] == [4, 0, 2]
    # every sync updates the three ranges left to right on both ranks; the owner of each gBest
    # (and only it) hands out its own row: g=4 -> rank 1 row 1, g=0 -> rank 0 row 0, g=2 -> rank 0 row 2
    ranges = [["range", 0, 88], ["range", 88, 176], ["range", 176, 257]]
    assert res[0]["log"] == ranges + [["row", 0]] + ranges + [["row", 2]] + ranges
    assert res[1]["log"] == [["row", 1]] + ranges + ranges + ranges


def test_shard_ownership_and_traffic():
    from paper_2009_03816_b200 import sharded
    assert sharded.owner_of(0, [3, 2]) == (0, 0) and sharded.owner_of(3, [3, 2]) == (1, 0)
    assert sharded.owner_of(7, [1] * 8) == (7, 0) and sharded.first_index(2, [3, 1, 4]) == 4
    t = sharded.bytes_received_per_sync(11_173_962, [2] * 8)
    assert t["gbest_broadcast"] == 4 * 11_173_962 and t["gather_all_particles"] == 4 * 11_173_962 * 14
    assert t["losses_all_gather"] == 64
    assert sharded.range_bounds(10, 3, 4) == [(0, 4), (4, 8), (8, 10)]
    assert sharded.range_bounds(11_173_962, 6) == [(i * 1_862_656, min(11_173_962, (i + 1) * 1_862_656))
                                                   for i in range(6)]
    assert sharded.range_bounds(100, 6) == [(0, 100)]
