#!/usr/bin/env python
"""Benchmark of the PSO-PS synchronisation stage on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4]
    python bench.py --impl reference ...        # the CPU oracle, same metric

One step = one pass of the synchronisation stage over the whole swarm: hand in
the K losses, selection kernel, fused update kernel (psops_set_losses +
psops_sync).  The metric is particle-elements updated per second; the roofline
object relates the fused update kernel's algorithmic bytes to the measured HBM
copy bandwidth of this machine's B200s.  Rank 0 prints one JSON line.

The line certifies what it timed: after the timed region the state the GPU was
left with is compared, on a seeded sample of columns, with the CPU oracle run
from the same initial state through the same number of syncs ("parity"); a
mismatch sets "parity_ok": false, is reported on stderr and makes the exit
status non-zero.  The oracle never runs inside a timed region.
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

# DRAM traffic of the fused update kernel from an ncu capture of a small case
# (N = 4 M, state larger than L2), per particle-element -- every value is
# touched once, so traffic grows in proportion to K x N -- and the hash of the
# source it was taken from: everything in psops_kernels.cuh up to the end of the
# update kernel, i.e. that kernel and all it uses.  The benchmark reports null
# once that text has changed, and for workloads whose state is kept in L2.
NCU_TRAFFIC = {"source_sha256": "8a56c0c1a46a1f7c167811c1992ddba1753b9dd1379854339f3eecaa9faa6245",
               "bytes_per_particle_element": 19.56,       # 2.505 / 2.503 GB per launch over 128 M: cfg4 recipe at N = 4 M
               "profile": "profiles/update_kernel_cfg4_n4m.txt"}
KERNEL_SOURCE = os.path.join(ROOT, "paper_2009_03816_b200", "csrc", "psops_kernels.cuh")
HASH_UNTIL = "// gBest snapshot for launches of kernel (b)"


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
    ap.add_argument("--min-seconds", type=float, default=0.25,
                    help="after the K timed steps, repeat K-step windows until this much device time has been "
                         "measured in total (their spread is reported; the headline uses the first K steps)")
    ap.add_argument("--parity", choices=["on", "off"], default="on",
                    help="compare the timed state with the CPU oracle on a column sample")
    ap.add_argument("--pieces", type=int, default=6, help="--parallelism shards: ranges of the gBest broadcast")
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


def workload_config(w, replicas_count):
    """The `config` object of the JSON line: names the workload; the same for
    the GPU arm and for the reference arm (whose bounded sample is described in
    its `cpu_baseline.sample`)."""
    return {"workload": f"{w.name}: K={w.K} particles x N={w.N} fp32 ({w.note}), "
                        f"omega={w.omega}, c1={w.c1}, c2={w.c2}, lambda={w.lam}, seed={w.seed}",
            "K": w.K, "N": w.N, "ld": w.ld, "replicas": replicas_count,
            "l2": "state (12*K*N bytes) exceeds L2; no flush needed" if 12 * w.K * w.N > (126 << 20)
                  else "state fits L2: an L2-resident result, reported as such",
            "parallelism": "replicas only"}


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
def device_state(w, dev, cols=None):
    """Upload the seeded recipe row by row: (x, v, pbest) as (K, ld) tensors.
    With `cols` also returns the initial (x, v) at those columns as numpy
    arrays, taken from the host rows before they are uploaded."""
    import torch
    from paper_2009_03816_b200 import workloads
    dx = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    dv = torch.zeros((w.K, w.ld), dtype=torch.float32, device=dev)
    xs = np.zeros((w.K, 0 if cols is None else cols.size), np.float32)
    vs = np.zeros_like(xs)
    for k in range(w.K):
        row = workloads.x_row(w, k)
        if cols is not None:
            xs[k] = row[cols]
        dx[k, :w.N] = torch.from_numpy(row).to(dev)
        if w.sigma_v != 0.0:
            row = workloads.v_row(w, k)
            if cols is not None:
                vs[k] = row[cols]
            dv[k, :w.N] = torch.from_numpy(row).to(dev)
    if cols is None:
        return dx, dv, dx.clone()
    return dx, dv, dx.clone(), xs, vs


def make_swarm(w, dev, flags=0, cols=None):
    from paper_2009_03816_b200 import binding
    dx, dv, dp, *sample = device_state(w, dev, cols)
    sw = binding.Swarm(dx, dv, dp, N=w.N, m_max=w.omega, m_min=w.omega, c1=w.c1, c2=w.c2,
                       seed=w.seed, flags=flags)
    sw.initial_sample = tuple(sample) if sample else None
    return sw


class Timing:
    """Device times of one timed region (CUDA events on the current stream)."""

    def __init__(self, seconds, step_ms=None):
        self.seconds = seconds                # first event to last event: the K steps of the contract
        self.step_ms = step_ms                # per-step durations, when every step had its own event pair
        self.window_ms_per_step = []          # further K-step windows, if any

    def stats(self, steps):
        out = {"ms_per_step_mean": self.seconds * 1e3 / steps}
        if self.step_ms:
            a = np.asarray(self.step_ms)
            out["per_step_ms"] = {"median": float(np.median(a)), "min": float(a.min()), "max": float(a.max()),
                                  "n": int(a.size)}
        if self.window_ms_per_step:
            a = np.asarray([self.seconds * 1e3 / steps] + self.window_ms_per_step)
            out["window_ms_per_step"] = {"median": float(np.median(a)), "min": float(a.min()),
                                         "max": float(a.max()), "n": int(a.size)}
        return out


def time_region(fn, steps, warmup, ranks, sampler=None, counter=None, per_step=False, min_seconds=0.0,
                first=0):
    """Warm up, then time exactly `steps` calls of fn(i) between barriers and
    device synchronisation, with CUDA events on the current stream (one pair
    around the region; with per_step one event between any two steps as well).
    If that measured less than min_seconds, further windows of `steps` calls
    follow (each between its own event pair) until the total reaches it.
    Returns (Timing, calls made, counter advance inside the first region)."""
    import torch
    from paper_2009_03816_b200 import replicas
    i = first
    for _ in range(warmup):
        fn(i)
        i += 1
    torch.cuda.synchronize()
    replicas.barrier(ranks)
    torch.cuda.synchronize()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1 if per_step else 2)]
    ctx = sampler if sampler is not None else _Null()
    c0 = counter() if counter is not None else 0
    with ctx:
        marks[0].record()
        for k in range(steps):
            fn(i)
            i += 1
            if per_step:
                marks[k + 1].record()
        if not per_step:
            marks[1].record()
        torch.cuda.synchronize()
        c1 = counter() if counter is not None else 0
        replicas.barrier(ranks)
        timing = Timing(marks[0].elapsed_time(marks[-1]) * 1e-3,
                        [marks[k].elapsed_time(marks[k + 1]) for k in range(steps)] if per_step else None)
        total = replicas.max_over_ranks(ranks, timing.seconds)
        while total < min_seconds and len(timing.window_ms_per_step) < 64:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                fn(i)
                i += 1
            e1.record()
            torch.cuda.synchronize()
            sec = e0.elapsed_time(e1) * 1e-3
            # every rank must make the same number of windows: agree on the slowest total
            total = replicas.max_over_ranks(ranks, total + sec) if ranks.world > 1 else total + sec
            timing.window_ms_per_step.append(sec * 1e3 / steps)
    return timing, i - first, c1 - c0


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


PARITY_COLUMNS = 4096       # random columns of the sample (plus every residue mod 1024, block edges, head and tail)
PARITY_TAIL = 8             # further syncs after the timed region whose selection is compared one by one


def time_sync_workload(w, dev, steps, warmup, ranks, sampler=None, fused_fitness=False, per_step=False,
                       min_seconds=0.0, cols=None, flags=0):
    """Time psops_set_losses + psops_sync on a fresh swarm of recipe `w`.
    Returns (swarm, Timing, syncs made since the initial state, launches in the
    first timed region, tensors to keep alive, device loss table)."""
    import torch
    from paper_2009_03816_b200 import binding, workloads
    flags |= binding.PSOPS_QUADRATIC if fused_fitness else 0
    sw = make_swarm(w, dev, flags, cols)
    keep = dtable = None
    if fused_fitness:
        d, t = workloads.quadratic_vectors(w)
        keep = (torch.from_numpy(d).to(dev), torch.from_numpy(t).to(dev))
        sw.set_quadratic(*keep)
        sw.eval_quadratic()

        def step(i):
            sw.sync(0, w.lam)
    else:
        dtable = torch.from_numpy(workloads.losses(w)).to(dev)

        def step(i):
            sw.set_losses(dtable[i % dtable.shape[0]])
            sw.sync(0, w.lam)
    timing, made, launches = time_region(step, steps, warmup, ranks, sampler, counter=lambda: sw.launches,
                                         per_step=per_step, min_seconds=min_seconds)
    return sw, timing, made, launches, keep, dtable


def _rel_err(got, want):
    """(max relative error, elements outside 1e-6, elements not bit-identical)
    under the parity contract |gpu - ref| <= 1e-6 max(|ref|, 1e-6 RMS(ref))."""
    rms = float(np.sqrt(np.mean(np.square(want, dtype=np.float64)))) if want.size else 0.0
    scale = np.maximum(np.abs(want).astype(np.float64), 1e-6 * rms if rms > 0 else 1e-300)
    same = (got.view(np.uint32) == want.view(np.uint32)) | ((got == 0) & (want == 0)) \
        | (np.isnan(got) & np.isnan(want))
    with np.errstate(invalid="ignore", over="ignore"):
        err = np.abs(got.astype(np.float64) - want.astype(np.float64)) / scale
    err = np.where(same, 0.0, err)
    err = np.where(np.isnan(err), np.inf, err)            # a NaN on one side only is a mismatch
    return float(err.max()) if err.size else 0.0, int((err > 1e-6).sum()), int((~same).sum())


def parity_after_timing(w, sw, made, cols, dtable, dev):
    """Follow the sampled columns through the same `made` syncs in the CPU
    oracle (outside any timed region) and compare with the state the GPU is
    in; then PARITY_TAIL further syncs on both sides with the selection
    compared after each."""
    import torch
    import oracle
    from paper_2009_03816_b200 import workloads
    xs, vs = sw.initial_sample
    table = workloads.losses(w)
    ref = oracle.RefSwarm(xs, vs, xs, m_max=w.omega, m_min=w.omega, t_max=1, c1=w.c1, c2=w.c2, seed=w.seed,
                          elem_index=cols, nthreads=os.cpu_count() or 1)
    for i in range(made):
        ref.sync(table[i % table.shape[0]], 0, w.lam)
    dcols = torch.from_numpy(cols).to(dev)

    def selection_mismatch():
        g, improved, pl = sw.info()
        return int(g != ref.g or not np.array_equal(improved, ref.improved)
                   or not np.array_equal(pl.view(np.uint32), ref.pbest_loss.view(np.uint32)))

    def state():
        worst, outside, inexact = 0.0, 0, 0
        for t, want in ((sw.x, ref.x), (sw.v, ref.v), (sw.pbest, ref.p)):
            e, o, n = _rel_err(t[:, dcols].cpu().numpy(), want)
            worst, outside, inexact = max(worst, e), outside + o, inexact + n
        return worst, outside, inexact

    mism = selection_mismatch()
    worst, outside, inexact = state()
    for j in range(PARITY_TAIL):
        i = made + j
        sw.set_losses(dtable[i % dtable.shape[0]])
        sw.sync(0, w.lam)
        ref.sync(table[i % table.shape[0]], 0, w.lam)
        mism += selection_mismatch()
    e2, o2, n2 = state()
    return {"ok": mism == 0 and outside + o2 == 0, "selection_mismatches": mism,
            "max_rel_err": max(worst, e2), "outside_1e-6": outside + o2, "inexact": inexact + n2,
            "columns": int(cols.size), "syncs": made + PARITY_TAIL,
            "checked": f"x, v, pbest at the sampled columns after the {made} syncs made since the initial state "
                       f"(warm-up, timed steps and windows) and again after {PARITY_TAIL} more; selection "
                       f"(g, improved mask, pBest_loss) bit for bit after the last timed sync and after each of "
                       f"the {PARITY_TAIL} (every earlier selection shaped the compared state)",
            "oracle": "oracle/psops_ref.c, same initial state, same loss table"}


def parity_fused_fitness(w, sw, keep, dev):
    """cfg5-style rows: the losses come from the device, so the oracle needs the
    whole swarm.  Take the state the timed region left, run ONE more sync on
    both sides (oracle on all host cores) and compare the losses it consumed,
    the selection, the new losses (bit for bit) and every element."""
    import torch
    import oracle
    nthreads = os.cpu_count() or 1
    N = w.N
    x, v, p = (t[:, :N].cpu().numpy() for t in (sw.x, sw.v, sw.pbest))
    d, t = (k.cpu().numpy() for k in keep)
    _, pl = sw.state()
    loss_gpu = sw.losses()
    loss_ref = oracle.quadratic_losses(x, d, t, nthreads=nthreads)
    mism = int(not np.array_equal(loss_gpu.view(np.uint32), loss_ref.view(np.uint32)))
    step, _ = sw.state()
    ref = oracle.RefSwarm(x, v, p, m_max=w.omega, m_min=w.omega, t_max=1, c1=w.c1, c2=w.c2, seed=w.seed,
                          nthreads=nthreads)
    ref.pbest_loss[:] = pl
    ref.s = step
    del x, v, p
    sw.sync(0, w.lam)
    ref.sync(loss_ref, 0, w.lam)
    g, improved, pl2 = sw.info()
    mism += int(g != ref.g or not np.array_equal(improved, ref.improved)
                or not np.array_equal(pl2.view(np.uint32), ref.pbest_loss.view(np.uint32)))
    new_ref = oracle.quadratic_losses(ref.x, d, t, nthreads=nthreads)
    mism += int(not np.array_equal(sw.losses().view(np.uint32), new_ref.view(np.uint32)))
    worst, outside, inexact = 0.0, 0, 0
    for tdev, want in ((sw.x, ref.x), (sw.v, ref.v), (sw.pbest, ref.p)):
        for k in range(w.K):                    # row by row keeps the host copies small
            e, o, n = _rel_err(tdev[k, :N].cpu().numpy(), want[k])
            worst, outside, inexact = max(worst, e), outside + o, inexact + n
    return {"ok": mism == 0 and outside == 0, "selection_mismatches": mism, "max_rel_err": worst,
            "outside_1e-6": outside, "inexact": inexact, "columns": int(N), "syncs": 1,
            "checked": "one further sync from the state the timed region left, whole swarm in the oracle: the "
                       "device-evaluated losses before and after it bit for bit, selection, every element of "
                       "x, v, pbest"}


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
    check = args.parity == "on" and ranks.is_root
    cols = workloads.sample_columns_dense(w.N, PARITY_COLUMNS, w.seed) if check and not fused else None
    sw, timing, made, launches, keep, dtable = time_sync_workload(
        w, dev, args.steps, args.warmup, ranks, sampler, fused, per_step=pe >= 50_000_000,
        min_seconds=args.min_seconds, cols=cols)
    seconds = timing.seconds
    rate, slowest = replicas.whole_job_rate(ranks, pe * args.steps, seconds)
    ms_per_step = slowest * 1e3 / args.steps
    achieved = sync_bytes(w, fused) / (seconds / args.steps) / 1e9
    parity = None
    if check:
        parity = parity_fused_fitness(w, sw, keep, dev) if fused else parity_after_timing(w, sw, made, cols, dtable, dev)

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
        "config": workload_config(w, ranks.world),
        "timing": timing.stats(args.steps),
        "clocks": sampler.report(),
        "e2e": e2e,
        "gpu_launches": int(replicas.sum_over_ranks(ranks, launches)),
        "roofline": {"bound": "hbm", "kernel": "psops_update_kernel", "achieved": achieved,
                     "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "bytes_per_launch": sync_bytes(w, fused), "traffic": ncu_traffic(w),
                     "note": "duration = timed region / steps (includes the selection kernel); the peak is a "
                             "measured 1:1 copy, which this 3:2 read:write kernel can exceed slightly -- "
                             "frac_of_nominal_8TBs is the fraction of the nominal HBM3e rate"},
        "parity": parity,
        "parity_ok": None if parity is None else bool(parity["ok"]),
    }
    sw.close()
    del sw, keep
    torch.cuda.empty_cache()

    if ranks.is_root and ranks.world == 1:
        if args.rows == "all":
            out["rows"] = other_rows(args, dev, ranks, peak)
            bad = [k for k, r in out["rows"].items() if isinstance(r, dict) and r.get("parity") and not r["parity"]["ok"]]
            if bad:
                out["parity_ok"] = False
                out["parity_failed_rows"] = bad
        if args.cpu_baseline == "on":
            out["cpu_baseline"] = cpu_baseline(w)
    if ranks.is_root:
        print(json.dumps(out), flush=True)
        if out["parity_ok"] is False:
            print("PARITY FAILURE: the timed state does not match the oracle: "
                  + json.dumps({"headline": parity, "rows": out.get("parity_failed_rows")}), file=sys.stderr, flush=True)
    replicas.finish(ranks)
    if out["parity_ok"] is False:
        raise SystemExit(3)


def run_shards(args, w, dev, dev_index, ranks, peak, peak_src):
    """One swarm, K / world particles per rank.  Per sync every rank receives
    4 K bytes of losses and 4 N bytes of gBest instead of the other ranks' rows;
    the broadcast travels in --pieces element ranges and the update of a range
    runs while the next one is on the wire."""
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
    drv = sharded.ShardedSync(sharded.swarm_engine(sw), counts, w.N, dev, pieces=args.pieces)
    table = torch.from_numpy(workloads.losses(w)).to(dev)
    sampler = ClockSampler(dev_index)

    def step(i):
        drv.sync(table[i % table.shape[0], first:first + n_here], 0, w.lam)

    timing, made, launches = time_region(step, args.steps, args.warmup, ranks, sampler,
                                         counter=lambda: sw.launches)
    # the phases of a sync, from a second short pass with an event between them (the events cost host
    # time, so they stay out of the timed region above)
    drv.timing = True
    for i in range(made, made + 20):
        step(i)
    phases = drv.timings_ms()
    seconds = timing.seconds
    slowest = replicas.max_over_ranks(ranks, seconds)
    bytes_here = 20 * n_here * w.N + 4 * w.N
    achieved = bytes_here / (seconds / args.steps) / 1e9
    phases = {k: (replicas.max_over_ranks(ranks, v) if isinstance(v, float) else v) for k, v in phases.items()}
    out = {
        "metric": METRIC, "value": w.K * w.N * args.steps / slowest, "unit": UNIT, "n_gpus": ranks.world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": slowest * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": f"{w.name}: K={w.K} particles x N={w.N} fp32 ({w.note}), one swarm sharded by particle",
                   "K": w.K, "N": w.N, "ld": w.ld, "particles_per_rank": n_here,
                   "parallelism": f"particle shards x{ranks.world}", "broadcast_pieces": len(drv.bounds),
                   "exchange_bytes_per_rank_per_sync": sharded.bytes_received_per_sync(w.N, counts)},
        "phases_ms_per_sync_max_over_ranks": phases,
        "clocks": sampler.report(), "e2e": None,
        "gpu_launches": int(replicas.sum_over_ranks(ranks, launches)),
        "roofline": {"bound": "hbm", "kernel": "psops_update_kernel", "achieved": achieved, "peak": peak,
                     "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                     "bytes_per_launch": bytes_here, "traffic": None,
                     "note": "duration = timed region / steps: collectives, selection (with the host's read of g) "
                             "and update of this rank's particles"},
    }
    sw.close()
    if ranks.is_root:
        print(json.dumps(out), flush=True)
    replicas.finish(ranks)


def ncu_traffic(w):
    if not NCU_TRAFFIC["source_sha256"] or update_kernel_source_sha256() != NCU_TRAFFIC["source_sha256"]:
        return None
    if 4 * w.K * w.N <= 0.52 * (126 << 20):       # an array is kept in L2: DRAM traffic is not proportional
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


def _row(w, timing, steps, nbytes, peak, K_here=None, parity=None):
    sec = timing.seconds
    gbs = nbytes / (sec / steps) / 1e9
    out = {"ms_per_step": sec * 1e3 / steps, "value": (K_here or w.K) * w.N * steps / sec, "unit": UNIT,
           "GBps": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0, "timing": timing.stats(steps)}
    if parity is not None:
        out["parity"] = parity
    return out


def time_variant(w, dev, ranks, peak, flags=0, shard=None, steps=100, min_seconds=0.05):
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
    timing, _, _ = time_region(step, steps, 5, ranks, per_step=True, min_seconds=min_seconds)
    out = _row(w, timing, steps, 20 * K_here * w.N + 4 * w.N, peak, K_here)
    sw.close()
    del sw
    torch.cuda.empty_cache()
    return out


def other_rows(args, dev, ranks, peak):
    """The remaining rows of the path, timed the same way (device-resident)."""
    import torch
    from paper_2009_03816_b200 import workloads
    rows = {}
    check = args.parity == "on"
    try:
        w3, w5 = workloads.CONFIGS["cfg3"], workloads.CONFIGS["cfg5"]
        if args.n:
            w3, w5 = w3.scaled(N=args.n), w5.scaled(N=args.n)
        S3, S5, W = args.row_steps or 100, args.row_steps or 50, (5 if not args.row_steps else 3)
        cols = workloads.sample_columns_dense(w3.N, PARITY_COLUMNS, w3.seed) if check else None
        sw, timing, made, _, _, dtable = time_sync_workload(w3, dev, S3, W, ranks, per_step=True,
                                                            min_seconds=0.0 if args.row_steps else 0.1, cols=cols)
        par = parity_after_timing(w3, sw, made, cols, dtable, dev) if check else None
        rows["cfg3_sync"] = _row(w3, timing, S3, sync_bytes(w3), peak, parity=par)
        timing, _, _ = time_region(lambda i: sw.average(), S3, W, ranks, per_step=True)
        rows["cfg3_average"] = _row(w3, timing, S3, average_bytes(w3), peak)
        if check:       # every row of x must now hold the same values: spot-check against row 0
            rows["cfg3_average"]["rows_equal"] = bool(torch.equal(sw.x[0, :w3.N], sw.x[w3.K - 1, :w3.N]))
        # SSGD baseline on the same rows: K gradient rows in, K weight rows out
        grad = torch.randn((w3.K, w3.ld), device=dev, generator=torch.Generator(device=dev).manual_seed(3))
        timing, _, _ = time_region(lambda i: sw.ssgd(grad, -0.01), S3, W, ranks, per_step=True)
        rows["cfg3_ssgd"] = _row(w3, timing, S3, 8 * w3.K * w3.N + 4 * w3.N, peak)
        del grad
        sw.close()
        del sw
        torch.cuda.empty_cache()
        short = 0.0 if args.row_steps else 0.05          # profiling captures want few launches
        rows["cfg3_sync_gbest_history"] = time_variant(w3, dev, ranks, peak, flags=4, steps=S3, min_seconds=short)
        # what one GPU of an 8-GPU particle-sharded run does per sync: 2 of the 16 particles,
        # gBest read from a broadcast buffer (the collectives themselves need more than one GPU)
        rows["cfg3_shard_2_of_16"] = time_variant(w3, dev, ranks, peak, shard=(0, 2), steps=S3, min_seconds=short)
        sw, timing, _, _, keep, _ = time_sync_workload(w5, dev, S5, W, ranks, fused_fitness=True, per_step=True)
        par = parity_fused_fitness(w5, sw, keep, dev) if check else None
        rows["cfg5_sync_fused_fitness"] = _row(w5, timing, S5, sync_bytes(w5, True), peak, parity=par)
        timing, _, _ = time_region(lambda i: sw.eval_quadratic(), S5, W, ranks, per_step=True)
        tiles = (w5.N + 127) // 128
        rows["cfg5_fitness_only"] = _row(w5, timing, S5, 4 * w5.K * w5.N + 8 * w5.N + 16 * w5.K * tiles, peak)
        sw.close()
        del sw, keep
        torch.cuda.empty_cache()
        # small swarms: cfg1, cfg2, and the paper's own regime of many workers on a LeNet-sized vector
        # (the cfg3 / cfg4 recipes with 16 / 32 particles at cfg1's 61,706 elements)
        small = {"cfg1": workloads.CONFIGS["cfg1"], "cfg2": workloads.CONFIGS["cfg2"],
                 "k16_n61706": workloads.CONFIGS["cfg3"].scaled(N=61_706),
                 "k32_n61706": workloads.CONFIGS["cfg4"].scaled(N=61_706)}
        for name, ws in (() if args.n else small.items()):
            cols = workloads.sample_columns_dense(ws.N, PARITY_COLUMNS, ws.seed) if check else None
            # no further windows here: cfg2's omega = 0.9, c = 2 lies outside PSO's stability region, and a
            # few hundred syncs beyond its 50 would overflow fp32 and leave nothing finite to compare
            sw, timing, made, launches, _, dtable = time_sync_workload(ws, dev, 200, 10, ranks, cols=cols)
            st = timing.stats(200)
            rows[name + "_sync"] = {"us_per_step": timing.seconds / 200 * 1e6, "value": ws.K * ws.N * 200 / timing.seconds,
                                    "unit": UNIT, "launches_per_sync": launches / 200,
                                    "GBps": sync_bytes(ws) / (timing.seconds / 200) / 1e9,
                                    "note": "small case: host launch rate / L2-resident", "timing": st,
                                    "us_per_step_cuda_graph": graph_us_per_sync(ws, dev)}
            if check:
                rows[name + "_sync"]["parity"] = parity_after_timing(ws, sw, made, cols, dtable, dev)
            sw.close()
            del sw
    except Exception as exc:  # report, do not lose the headline line
        import traceback
        rows["error"] = repr(exc) + " | " + traceback.format_exc().splitlines()[-3].strip()
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


def _time_oracle(w, nthreads, target_seconds, syncs):
    n_cols = 1 << 14
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
    return w.K * n_cols * syncs / sec, n_cols, sec


def cpu_baseline(w, target_seconds=1.5, syncs=3):
    """Time the oracle as it stands on this machine's host cores on a bounded
    sample of the workload's columns: all cores (OpenMP over elements) and one
    thread."""
    nthreads = os.cpu_count() or 1
    value, n_cols, sec = _time_oracle(w, nthreads, target_seconds, syncs)
    value1, n_cols1, sec1 = _time_oracle(w, 1, target_seconds, syncs)
    return {"value": value, "unit": UNIT, "cores": nthreads, "kind": "oracle",
            "sample": f"{syncs} syncs of the first {n_cols} of {w.N} columns, all K={w.K} particles, "
                      f"OpenMP over elements", "seconds": sec,
            "one_thread": {"value": value1, "cores": 1, "seconds": sec1,
                           "sample": f"{syncs} syncs of the first {n_cols1} of {w.N} columns"}}


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
        "config": workload_config(w, args.gpus),
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
