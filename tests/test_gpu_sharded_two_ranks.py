"""The particle-sharded sync as two real ranks: two processes, each with its own
context, rows and CUDA stream, exchanging the losses and the chunked gBest
broadcast through torch.distributed.  Only one GPU is needed: both ranks use
cuda:0 and rendezvous over gloo (which stages CUDA tensors through the host);
no kernel of one rank waits for a kernel of the other -- all waiting is done
by the hosts inside the collectives.  Every rank runs the oracle on the whole
swarm and compares its own rows after every sync."""
import json
import os
import socket
import subprocess
import sys
import textwrap

import pytest

from conftest import ROOT

pytestmark = pytest.mark.gpu

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, os.environ["PSOPS_ROOT"]); sys.path.insert(0, os.path.join(os.environ["PSOPS_ROOT"], "tests"))
    import numpy as np, torch
    import oracle
    from paper_2009_03816_b200 import binding, replicas, sharded
    from paper_2009_03816_b200 import build as _build
    r = replicas.init_from_env(backend="gloo")
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    counts = json.loads(os.environ["PSOPS_COUNTS"])
    K, N = sum(counts), 50_003
    ld = (N + 1023) // 1024 * 1024
    rng = np.random.default_rng(21)
    x = rng.standard_normal((K, N)).astype(np.float32)
    v = (0.1 * rng.standard_normal((K, N))).astype(np.float32)
    p = (x + 0.5 * rng.standard_normal((K, N))).astype(np.float32)
    ref = oracle.RefSwarm(x, v, p, m_max=0.9, m_min=0.3, t_max=40, c1=0.2, c2=0.9, seed=31, nthreads=2)
    first, n = sharded.first_index(r.rank, counts), counts[r.rank]
    def rows(a):
        t = torch.zeros((n, ld), dtype=torch.float32, device=dev)
        t[:, :N] = torch.from_numpy(a[first:first + n]).to(dev)
        return t
    dx, dv, dp = rows(x), rows(v), rows(p)
    _build.build_library()
    sw = binding.Swarm(dx, dv, dp, N=N, m_max=0.9, m_min=0.3, t_max=40, c1=0.2, c2=0.9, seed=31,
                       k_first=first, K_total=K)
    drv = sharded.ShardedSync(sharded.swarm_engine(sw), counts, N, dev, pieces=3)
    assert len(drv.bounds) == 3
    owners = []
    table = rng.random((6, K)).astype(np.float32)
    table[2, K - 1] = 0.0                      # gBest on the last rank ...
    table[3, 0] = 0.0                          # ... and on the first
    for s in range(6):
        mine = torch.from_numpy(table[s, first:first + n].copy()).to(dev)
        g = drv.sync(mine, 4 * s, 1.0 + s)
        ref.sync(table[s], 4 * s, 1.0 + s)
        assert g == ref.g, (s, g, ref.g)
        owners.append(sharded.owner_of(g, counts)[0])
        gi, improved, pl = sw.info()
        assert gi == ref.g and np.array_equal(improved, ref.improved)
        assert np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32))
        for t, want in ((dx, ref.x), (dv, ref.v), (dp, ref.p)):
            got = t[:, :N].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), want[first:first + n].view(np.uint32)), (r.rank, s)
        assert torch.all(dx[:, N:] == 0)
    sw.close()
    print(json.dumps({"rank": r.rank, "owners": owners}))
    replicas.finish(r)
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("counts", [[2, 2], [3, 2]])       # equal shards: one collective for the losses; unequal: padded
def test_two_sharded_ranks_on_one_gpu_match_the_oracle(tmp_path, counts):
    script = tmp_path / "shard_rank.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), PSOPS_ROOT=ROOT, PSOPS_COUNTS=json.dumps(counts), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-3000:]
    res = [json.loads(o[0].strip().splitlines()[-1]) for o in outs]
    assert res[0]["owners"] == res[1]["owners"]
    assert set(res[0]["owners"]) == {0, 1}                 # both ranks were the source of a broadcast
