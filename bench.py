#!/usr/bin/env python
"""Benchmark of the PSO-PS synchronisation stage on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4]
    python bench.py --impl reference ...        # the CPU oracle, same metric

One step = one pass of the synchronisation stage over the whole swarm: hand in
the K losses, selection kernel, fused update kernel (psops_set_losses +
psops_sync).  The metric is particle-elements updated per second; the roofline
object relates the fused update kernel's algorithmic bytes to the measured HBM
copy bandwidth of this machine's B200s.  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pso_sync_throughput"
UNIT = "particle-elements/s"
FALLBACK_HBM_GBS = 6650.0           # earlier measurement on this machine, used only if no measured file

# DRAM traffic of the fused update kernel from an ncu capture, per
# particle-element, and the hash of the source it was taken from: everything in
# psops_kernels.cuh up to the averaging kernel, i.e. the update kernel and all
# it uses.  The benchmark reports null once that text has changed.
NCU_TRAFFIC = {"source_sha256": "ada5eebaa22a962d5e61660f02521acb7dc8cc903445cbd8c4328c8b43ec14c5",
               "bytes_per_particle_element": 19.93,       # 16.30 GB / 817.8 M: full-size cfg4 launches, 1-pass counters
               "profile": "profiles/update_kernel_cfg4_n4m_full.txt"}
KERNEL_SOURCE = os.path.join(ROOT, "paper_2009_03816_b200", "csrc", "psops_kernels.cuh")
HASH_UNTIL = "// Kernel (c): parameter averaging"


def update_kernel_source_sha256() -> str:
    with open(KERNEL_SOURCE) as fh:
        text = fh.read()
    return hashlib.sha256(text[:text.index(HASH_UNTIL)].encode()).hexdigest()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["psops", "reference"], default="psops")
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--n", type=int, default=0,
                    help="run the workload's recipe at this vector length instead (profiling captures)")
    ap.add_argument("--e2e-steps", type=int, default=4, help="0 skips the host-buffer measurement")
    ap.add_argument("--rows", choices=["all", "none"], default="all",
                    help="also time the other rows of the path (averaging, cfg3, fused fitness)")
    ap.add_argument("--row-steps", type=int, default=0,
                    help="timed steps per extra row (default 100, 50 for cfg5); with --n for small captures")
    ap.add_argument("--cpu-baseline", choices=["on", "off"], default="on")
    ap.add_argument("--parallelism", choices=["replicas", "shards"], default="replicas",
                    help="shards: ONE swarm split by particle over the ranks (all-gather of losses + "
                         "broadcast of the best row per sync); strong scaling, not the default metric")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def sync_bytes(w, fused_fitness=False) -> int:
    """Algorithmic bytes of one sync: w, v read and written, pBest read or
    written (20 B per particle-element) plus one read of the gBest row."""
    b = 20 * w.K * w.N + 4 * w.N
    if fused_fitness:
        tiles = (w.N + 127) // 128
        b += 8 * w.N + 16 * w.K * tiles          # dvec, tvec; tile sums written then read
    return b


def average_bytes(w) -> int:
    return 8 * w.K * w.N


# ---------------------------------------------------------------------------
# Clock sampling (read-only NVML queries from a thread during the timed region)
# ---------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
        0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
        0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.samples, self.reason_bits = [], 0
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # pragma: no cover
            self.error = repr(exc)

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                try:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                except Exception:
                    pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.ok:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def report(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        reasons = [name for bit, name in self.REASONS.items()
                   if self.reason_bits & bit and name != "gpu_idle"]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.samples)}


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def device_state(w, dev):
    """Upload the seeded recipe row by row: (x, v, pbest) as (K, ld) tensors."""
    import torch
    from paper_2009_03816_b200 import workloads
    dx = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    dv = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    for k in range(w.K):
        dx[k, :w.N] = torch.from_numpy(workloads.x_row(w, k)).to(dev)
        if w.sigma_v != 0.0:
            dv[k, :w.N] = torch.from_numpy(workloads.v_row(w, k)).to(dev)
    return dx, dv, dx.clone()


def make_swarm(w, dev, flags=0):
    from paper_2009_03816_b200 import binding
    dx, dv, dp = device_state(w, dev)
    sw = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                       seed=w.seed, flags=flags)
    return sw


def time_region(fn, steps, warmup, ranks, sampler=None, counter=None):
    """Warm up, then time exactly `steps` calls of fn(i) between barriers and
    device synchronisation, with CUDA events on the current stream.  Returns
    this rank's elapsed seconds (and, with `counter`, how much that counter
    advanced inside the timed region)."""
    import torch
    from paper_2009_03816_b200 import replicas
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    replicas.barrier(ranks)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ctx = sampler if sampler is not None else _Null()
    c0 = counter() if counter is not None else 0
    with ctx:
        e0.record()
        for i in range(steps):
            fn(warmup + i)
        e1.record()
        torch.cuda.synchronize()
    c1 = counter() if counter is not None else 0
    replicas.barrier(ranks)
    seconds = e0.elapsed_time(e1) * 1e-3
    return (seconds, c1 - c0) if counter is not None else seconds


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def time_sync_workload(w, dev, steps, warmup, ranks, sampler=None, fused_fitness=False):
    import torch
    from paper_2009_03816_b200 import binding, workloads
    flags = binding.PSOPS_QUADRATIC if fused_fitness else 0
    sw = make_swarm(w, dev, flags)
    keep = None
    if fused_fitness:
        d, t = workloads.quadratic_vectors(w)
        keep = (torch.from_numpy(d).to(dev), torch.from_numpy(t).to(dev))
        sw.set_quadratic(*keep)
        sw.eval_quadratic()

        def step(i):
            sw.sync(0, w.lam)
    else:
        table = torch.from_numpy(workloads.losses(w)).to(dev)

        def step(i):
            sw.set_losses(table[i % table.shape[0]])
            sw.sync(0, w.lam)
    seconds, launches = time_region(step, steps, warmup, ranks, sampler, counter=lambda: sw.launches)
    return sw, seconds, launches, keep


def run_psops(args):
    import torch
    from paper_2009_03816_b200 import binding, replicas, workloads
    from paper_2009_03816_b200 import build as _build

    ranks = replicas.init_from_env()
    if ranks.world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={ranks.world}")
    _build.build_library() if ranks.local_rank == 0 else None
    replicas.barrier(ranks) if ranks.world > 1 else None
    binding.load()
    dev_index = ranks.local_rank % torch.cuda.device_count()    # replicas may share a GPU
    torch.cuda.set_device(dev_index)
    dev = torch.device("cuda", dev_index)
    w = workloads.CONFIGS[args.workload]
    if args.n:
        w = w.scaled(N=args.n)
    peak, peak_src = measured_peak()
    pe = w.K * w.N

    if args.parallelism == "shards":
        run_shards(args, w, dev, dev_index, ranks, peak, peak_src)
        return
    sampler = ClockSampler(dev_index)
    fused = w.quadratic
    sw, seconds, launches, keep = time_sync_workload(w, dev, args.steps, args.warmup, ranks, sampler, fused)
    rate, slowest = replicas.whole_job_rate(ranks, pe * args.steps, seconds)
    ms_per_step = slowest * 1e3 / args.steps
    achieved = sync_bytes(w, fused) / (seconds / args.steps) / 1e9

    # ---- end to end: host buffers in, host buffers out, through psops_sync_host
    e2e = None
    if args.e2e_steps > 0:
        table = workloads.losses(w) if not fused else None
        h_in = torch.empty((w.K, w.ld), dtype=torch.float32).pin_memory()
        h_out = torch.empty((w.K, w.ld), dtype=torch.float32).pin_memory()
        h_in.copy_(sw.x)
        hl = np.ascontiguousarray(table[0]) if table is not None else sw.losses()

        def e2e_step(i):
            sw.sync_host(h_in, hl if table is None else table[i % table.shape[0]], 0, w.lam, h_out)

        e2e_step(0)
        torch.cuda.synchronize()
        replicas.barrier(ranks)
        t0 = time.perf_counter()
        for i in range(args.e2e_steps):
            e2e_step(1 + i)
        torch.cuda.synchronize()
        e2e_seconds = time.perf_counter() - t0
        e2e_rate, _ = replicas.whole_job_rate(ranks, pe * args.e2e_steps, e2e_seconds)
        del h_in, h_out
        e2e = {"value": e2e_rate, "unit": UNIT, "h2d_bytes_per_step": 4 * w.K * w.N + 4 * w.K,
               "d2h_bytes_per_step": 4 * w.K * w.N, "steps": args.e2e_steps,
               "ms_per_step": e2e_seconds * 1e3 / args.e2e_steps,
               "call": "psops_sync_host (pinned host weights in, new weights out)"}

    out = {
        "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": ranks.world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: K={w.K} particles x N={w.N} fp32 ({w.note}), "
                               f"omega={w.omega}, c1={w.c1}, c2={w.c2}, lambda={w.lam}, seed={w.seed}",
                   "K": w.K, "N": w.N, "ld": w.ld, "replicas": ranks.world,
                   "l2": "state (12*K*N bytes) exceeds L2; no flush needed",
                   "parallelism": "replicas only"},
        "clocks": sampler.report(),
        "e2e": e2e,
        "gpu_launches": int(replicas.sum_over_ranks(ranks, launches)),
        "roofline": {"bound": "hbm", "kernel": "psops_update_kernel", "achieved": achieved,
                     "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "bytes_per_launch": sync_bytes(w, fused), "traffic": ncu_traffic(w),
                     "note": "duration = timed region / steps (includes the selection kernel)"},
    }
    sw.close()
    del sw, keep
    torch.cuda.empty_cache()

    if ranks.is_root and ranks.world == 1:
        if args.rows == "all":
            out["rows"] = other_rows(args, dev, ranks, peak)
        if args.cpu_baseline == "on":
            out["cpu_baseline"] = cpu_baseline(w)
    if ranks.is_root:
        print(json.dumps(out), flush=True)
    replicas.finish(ranks)


def run_shards(args, w, dev, dev_index, ranks, peak, peak_src):
    """One swarm, K / world particles per rank.  Per sync every rank receives
    4 K bytes of losses and 4 N bytes of gBest instead of the other ranks' rows."""
    import torch
    from paper_2009_03816_b200 import binding, replicas, sharded, workloads
    if w.K % ranks.world or w.quadratic:
        raise SystemExit("--parallelism shards needs K divisible by the ranks and a loss-table workload")
    n_here = w.K // ranks.world
    counts = [n_here] * ranks.world
    first = sharded.first_index(ranks.rank, counts)
    dx = torch.zeros((n_here, w.ld), dtype=torch.float32, device=dev)
    dv = torch.zeros((n_here, w.ld), dtype=torch.float32, device=dev)
    for r in range(n_here):
        dx[r, :w.N] = torch.from_numpy(workloads.x_row(w, first + r)).to(dev)
        if w.sigma_v != 0.0:
            dv[r, :w.N] = torch.from_numpy(workloads.v_row(w, first + r)).to(dev)
    sw = binding.Swarm(dx, dv, dx.clone(), N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                       seed=w.seed, k_first=first, K_total=w.K)
    drv = sharded.ShardedSync(sharded.swarm_engine(sw), counts, w.N, dev)
    table = torch.from_numpy(workloads.losses(w)).to(dev)
    sampler = ClockSampler(dev_index)

    def step(i):
        drv.sync(table[i % table.shape[0], first:first + n_here], 0, w.lam)

    seconds, launches = time_region(step, args.steps, args.warmup, ranks, sampler, counter=lambda: sw.launches)
    slowest = replicas.max_over_ranks(ranks, seconds)
    bytes_here = 20 * n_here * w.N + 4 * w.N
    achieved = bytes_here / (seconds / args.steps) / 1e9
    out = {
        "metric": METRIC, "value": w.K * w.N * args.steps / slowest, "unit": UNIT, "n_gpus": ranks.world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": slowest * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{w.name}: K={w.K} particles x N={w.N} fp32 ({w.note}), one swarm sharded by particle",
                   "K": w.K, "N": w.N, "ld": w.ld, "particles_per_rank": n_here,
                   "parallelism": f"particle shards x{ranks.world}",
                   "exchange_bytes_per_rank_per_sync": sharded.bytes_received_per_sync(w.N, counts)},
        "clocks": sampler.report(), "e2e": None,
        "gpu_launches": int(replicas.sum_over_ranks(ranks, launches)),
        "roofline": {"bound": "hbm", "kernel": "psops_update_kernel", "achieved": achieved, "peak": peak,
                     "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                     "bytes_per_launch": bytes_here, "traffic": None,
                     "note": "duration = timed region / steps: collectives, selection (with its host read of g) "
                             "and update of this rank's particles"},
    }
    sw.close()
    if ranks.is_root:
        print(json.dumps(out), flush=True)
    replicas.finish(ranks)


def ncu_traffic(w):
    if not NCU_TRAFFIC["source_sha256"] or update_kernel_source_sha256() != NCU_TRAFFIC["source_sha256"]:
        return None
    return NCU_TRAFFIC["bytes_per_particle_element"] * w.K * w.N


def graph_us_per_sync(w, dev, replays=20):
    """All S syncs of a small workload recorded into one CUDA graph (losses read
    from the device table, step counter kept on the device) and replayed:
    device time per sync without the host's launch cost."""
    import torch
    from paper_2009_03816_b200 import workloads
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        sw = make_swarm(w, dev)
        table = torch.from_numpy(workloads.losses(w)).to(dev)
    stream.synchronize()
    sw.close()
    from paper_2009_03816_b200 import binding
    sw = binding.Swarm(sw.x, sw.v, sw.pbest, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                       seed=w.seed, stream=stream.cuda_stream)
    rows = [table[s] for s in range(table.shape[0])]
    with torch.cuda.stream(stream):
        sw.set_losses(rows[0])
        sw.sync(0, w.lam)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for r in rows:
            sw.set_losses(r)
            sw.sync(0, w.lam)
    with torch.cuda.stream(stream):
        for _ in range(3):
            graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(replays):
            graph.replay()
        e1.record()
    stream.synchronize()
    sw.close()
    return e0.elapsed_time(e1) * 1e3 / (replays * len(rows))


def time_variant(w, dev, ranks, peak, flags=0, shard=None, steps=100):
    """psops_sync with a flag set, or the select + update pair of one particle shard."""
    import torch
    from paper_2009_03816_b200 import binding, workloads
    table = torch.from_numpy(workloads.losses(w)).to(dev)
    if shard is None:
        sw = make_swarm(w, dev, flags)
        K_here = w.K

        def step(i):
            sw.set_losses(table[i % table.shape[0]])
            sw.sync(0, w.lam)
    else:
        first, K_here = shard
        dx, dv, dp = device_state(w.with_particles(K_here), dev)
        sw = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                           seed=w.seed, k_first=first, K_total=w.K)
        gbest = dx[0].clone()

        def step(i):
            sw.set_losses(table[i % table.shape[0]])
            sw.shard_select()
            sw.shard_update(gbest, 0, w.lam)
    sec = time_region(step, steps, 5, ranks)
    gbs = (20 * K_here * w.N + 4 * w.N) / (sec / steps) / 1e9
    sw.close()
    del sw
    torch.cuda.empty_cache()
    return {"ms_per_step": sec * 1e3 / steps, "value": K_here * w.N * steps / sec, "unit": UNIT,
            "GBps": gbs, "frac": gbs / peak}


def other_rows(args, dev, ranks, peak):
    """The remaining rows of the path, timed the same way (device-resident)."""
    import torch
    from paper_2009_03816_b200 import workloads
    rows = {}
    try:
        w3, w5 = workloads.CONFIGS["cfg3"], workloads.CONFIGS["cfg5"]
        if args.n:
            w3, w5 = w3.scaled(N=args.n), w5.scaled(N=args.n)
        S3, S5, W = args.row_steps or 100, args.row_steps or 50, (5 if not args.row_steps else 3)
        sw, sec, _, _ = time_sync_workload(w3, dev, S3, W, ranks)
        gbs = sync_bytes(w3) / (sec / S3) / 1e9
        rows["cfg3_sync"] = {"ms_per_step": sec * 1e3 / S3, "value": w3.K * w3.N * S3 / sec, "unit": UNIT,
                             "GBps": gbs, "frac": gbs / peak}
        sec = time_region(lambda i: sw.average(), S3, W, ranks)
        gbs = average_bytes(w3) / (sec / S3) / 1e9
        rows["cfg3_average"] = {"ms_per_step": sec * 1e3 / S3, "value": w3.K * w3.N * S3 / sec, "unit": UNIT,
                                "GBps": gbs, "frac": gbs / peak}
        # SSGD baseline on the same rows: K gradient rows in, K weight rows out
        grad = torch.randn((w3.K, w3.ld), device=dev, generator=torch.Generator(device=dev).manual_seed(3))
        sec = time_region(lambda i: sw.ssgd(grad, -0.01), S3, W, ranks)
        gbs = (8 * w3.K * w3.N + 4 * w3.N) / (sec / S3) / 1e9
        rows["cfg3_ssgd"] = {"ms_per_step": sec * 1e3 / S3, "value": w3.K * w3.N * S3 / sec, "unit": UNIT,
                             "GBps": gbs, "frac": gbs / peak}
        del grad
        sw.close()
        del sw
        torch.cuda.empty_cache()
        rows["cfg3_sync_gbest_history"] = time_variant(w3, dev, ranks, peak, flags=4, steps=S3)
        # what one GPU of an 8-GPU particle-sharded run does per sync: 2 of the 16 particles,
        # gBest read from a broadcast buffer (the collectives themselves need more than one GPU)
        rows["cfg3_shard_2_of_16"] = time_variant(w3, dev, ranks, peak, shard=(0, 2), steps=S3)
        sw, sec, _, keep = time_sync_workload(w5, dev, S5, W, ranks, fused_fitness=True)
        gbs = sync_bytes(w5, True) / (sec / S5) / 1e9
        rows["cfg5_sync_fused_fitness"] = {"ms_per_step": sec * 1e3 / S5, "value": w5.K * w5.N * S5 / sec,
                                           "unit": UNIT, "GBps": gbs, "frac": gbs / peak}
        sec = time_region(lambda i: sw.eval_quadratic(), S5, W, ranks)
        tiles = (w5.N + 127) // 128
        gbs = (4 * w5.K * w5.N + 8 * w5.N + 16 * w5.K * tiles) / (sec / S5) / 1e9
        rows["cfg5_fitness_only"] = {"ms_per_step": sec * 1e3 / S5, "value": w5.K * w5.N * S5 / sec,
                                     "unit": UNIT, "GBps": gbs, "frac": gbs / peak}
        sw.close()
        del sw, keep
        torch.cuda.empty_cache()
        for name in (() if args.n else ("cfg1", "cfg2")):
            ws = workloads.CONFIGS[name]
            sw, sec, _, _ = time_sync_workload(ws, dev, 200, 10, ranks)
            rows[name + "_sync"] = {"us_per_step": sec / 200 * 1e6, "value": ws.K * ws.N * 200 / sec,
                                    "unit": UNIT, "note": "small case: host launch rate / L2-resident",
                                    "us_per_step_cuda_graph": graph_us_per_sync(ws, dev)}
            sw.close()
            del sw
    except Exception as exc:  # report, do not lose the headline line
        rows["error"] = repr(exc)
    return rows


# ---------------------------------------------------------------------------
# CPU oracle: reported baseline and the reference arm
# ---------------------------------------------------------------------------
def oracle_sample(w, n_cols, nthreads):
    import oracle
    from paper_2009_03816_b200 import workloads
    ws = w.scaled(N=n_cols)
    x, v, p = workloads.state(ws)
    ref = oracle.RefSwarm(x[:, :n_cols], v[:, :n_cols], p[:, :n_cols], m_max=w.omega, m_min=w.omega,
                          t_max=1, c1=w.c1, c2=w.c2, seed=w.seed, nthreads=nthreads)
    if w.quadratic:
        d, t = workloads.quadratic_vectors(ws)
        table = None
    else:
        d = t = None
        table = workloads.losses(ws)
    return ref, table, d, t


def oracle_step(ref, w, table, d, t, i, nthreads):
    import oracle
    if table is None:
        loss = oracle.quadratic_losses(ref.x, d, t, nthreads=nthreads)
    else:
        loss = table[i % table.shape[0]]
    ref.sync(loss, 0, w.lam)


def cpu_baseline(w, target_seconds=1.5, syncs=3):
    """Time the oracle as it stands on this machine's host cores on a bounded
    sample of the workload's columns."""
    nthreads = os.cpu_count() or 1
    n_cols = 1 << 16
    ref, table, d, t = oracle_sample(w, n_cols, nthreads)
    t0 = time.perf_counter()
    oracle_step(ref, w, table, d, t, 0, nthreads)
    probe = max(time.perf_counter() - t0, 1e-4)
    n_cols = int(min(w.N, max(n_cols, n_cols * target_seconds / probe)))
    ref, table, d, t = oracle_sample(w, n_cols, nthreads)
    t0 = time.perf_counter()
    for i in range(syncs):
        oracle_step(ref, w, table, d, t, i, nthreads)
    sec = time.perf_counter() - t0
    return {"value": w.K * n_cols * syncs / sec, "unit": UNIT, "cores": nthreads, "kind": "oracle",
            "sample": f"{syncs} syncs of the first {n_cols} of {w.N} columns, all K={w.K} particles, "
                      f"OpenMP over elements", "seconds": sec}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2009_03816_b200 import workloads
    w = workloads.CONFIGS[args.workload]
    nthreads = os.cpu_count() or 1
    n_cols = 1 << 16
    ref, table, d, t = oracle_sample(w, n_cols, nthreads)
    t0 = time.perf_counter()
    oracle_step(ref, w, table, d, t, 0, nthreads)
    probe = max(time.perf_counter() - t0, 1e-4)
    budget = 90.0 / max(1, args.steps + args.warmup)          # whole run within a few minutes
    n_cols = int(min(w.N, max(1024, n_cols * min(budget, 1.0) / probe)))
    ref, table, d, t = oracle_sample(w, n_cols, nthreads)
    for i in range(args.warmup):
        oracle_step(ref, w, table, d, t, i, nthreads)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle_step(ref, w, table, d, t, args.warmup + i, nthreads)
    sec = time.perf_counter() - t0
    value = w.K * n_cols * args.steps / sec
    sample = (f"each step = one sync of the first {n_cols} of {w.N} columns, all K={w.K} particles, "
              f"OpenMP over elements")
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{w.name}: K={w.K} particles x N={w.N} fp32 ({w.note}), "
                               f"omega={w.omega}, c1={w.c1}, c2={w.c2}, lambda={w.lam}, seed={w.seed}",
                   "K": w.K, "N": w.N, "sample_columns": n_cols},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": nthreads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_psops(a)
