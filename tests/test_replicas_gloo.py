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
