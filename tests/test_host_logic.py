"""CPU-only checks: the C-ABI library loads and exports what the header
declares, host-side validation answers before any CUDA call, the schedule
scalar agrees with the oracle, and the workload generators are deterministic."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from conftest import ROOT
from paper_2009_03816_b200 import binding, workloads
from paper_2009_03816_b200 import build as _build


@pytest.fixture(scope="module")
def lib():
    _build.build_library()
    return binding.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "psops.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(psops_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    declared = _declared_symbols()
    assert len(declared) >= 19
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == declared


def test_config_struct_layout_matches_header():
    # int32 K (+pad), int64 N, ld, 2 floats, int64 t_max, 2 floats, uint64 seed, uint32 flags (+pad)
    assert ctypes.sizeof(binding.psops_config) == 64
    assert binding.psops_config.N.offset == 8 and binding.psops_config.seed.offset == 48


def test_workspace_bytes(lib):
    base = binding.make_config(8, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    n0 = binding.psops_workspace_bytes(base)
    assert n0 > 0 and n0 % 256 == 0
    keep = binding.make_config(8, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1,
                               flags=binding.PSOPS_KEEP_GBEST)
    assert binding.psops_workspace_bytes(keep) >= n0 + 4000
    quad = binding.make_config(8, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1,
                               flags=binding.PSOPS_QUADRATIC)
    assert binding.psops_workspace_bytes(quad) >= n0 + 8 * 8 * 8      # K x ceil(N/128) doubles
    # many particles on few elements: the update may split the rows over more blocks and then keeps
    # a snapshot of the gBest row in the workspace -- by the swarm's shape alone, whatever the device
    many = binding.make_config(16, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    few = binding.make_config(8, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    big = binding.make_config(16, (1 << 19) + 4, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    assert binding.psops_workspace_bytes(many) >= binding.psops_workspace_bytes(few) + 4000
    assert binding.psops_workspace_bytes(big) == binding.psops_workspace_bytes(many) - 4096
    many_kept = binding.make_config(16, 1000, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1,
                                    flags=binding.PSOPS_KEEP_GBEST)
    assert binding.psops_workspace_bytes(many_kept) == binding.psops_workspace_bytes(many)   # one row serves both
    for bad in (dict(K=0), dict(K=1025), dict(N=0), dict(N=1 << 33), dict(ld=999), dict(t_max=0),
                dict(flags=16), dict(c1=float("nan")), dict(m_max=float("inf"))):
        kw = dict(K=8, N=1000, ld=1000, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=1, flags=0)
        kw.update(bad)
        K, N, ld = kw.pop("K"), kw.pop("N"), kw.pop("ld")
        assert binding.psops_workspace_bytes(binding.make_config(K, N, ld, **kw)) == 0, bad


def test_create_rejects_bad_arguments_before_touching_cuda(lib):
    good = binding.make_config(4, 100, 100, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    bad = binding.make_config(0, 100, 100, m_max=0.7, m_min=0.7, c1=1.5, c2=1.5, seed=1)
    fake = 0x10000                                                    # never dereferenced
    cases = [
        (bad, fake, fake, fake, fake, 1 << 20, binding.PSOPS_EINVAL),
        (good, 0, fake, fake, fake, 1 << 20, binding.PSOPS_EINVAL),
        (good, fake, fake, 0, fake, 1 << 20, binding.PSOPS_EINVAL),
        (good, fake + 2, fake, fake, fake, 1 << 20, binding.PSOPS_EALIGN),
        (good, fake, fake, fake, 0, 1 << 20, binding.PSOPS_EWORKSPACE),
        (good, fake, fake, fake, fake + 16, 1 << 20, binding.PSOPS_EWORKSPACE),
        (good, fake, fake, fake, fake, 8, binding.PSOPS_EWORKSPACE),
    ]
    for cfg, x, v, p, ws, nbytes, code in cases:
        with pytest.raises(binding.PsopsError) as e:
            binding.psops_create(cfg, x, v, p, ws, nbytes)
        assert e.value.code == code
    # null context everywhere
    null = ctypes.c_void_p()
    assert lib.psops_sync(null, 0, 1.0) == binding.PSOPS_EINVAL
    assert lib.psops_average(null) == binding.PSOPS_EINVAL
    assert lib.psops_set_losses(null, None, 0) == binding.PSOPS_EINVAL
    assert lib.psops_destroy(null) == binding.PSOPS_EINVAL
    assert lib.psops_launch_count(null) == 0


def test_static_fitness_validates_before_touching_cuda(lib):
    fake = 0x10000                                                    # never dereferenced
    f = lib.psops_quadratic_fitness_static
    assert f(None, 100, 2, 100, fake, fake, fake, None) == binding.PSOPS_EINVAL
    assert f(fake, 100, 2, 100, fake, fake, None, None) == binding.PSOPS_EINVAL
    assert f(fake, 99, 2, 100, fake, fake, fake, None) == binding.PSOPS_EINVAL      # ld < N
    assert f(fake, 100, 0, 100, fake, fake, fake, None) == binding.PSOPS_EINVAL
    assert f(fake + 1, 100, 2, 100, fake, fake, fake, None) == binding.PSOPS_EALIGN
    n = 128 * binding.PSOPS_STATIC_SCRATCH_DOUBLES
    assert f(fake, n, 2, n, fake, fake, fake, None) == binding.PSOPS_ELIMIT         # 2 * tiles > limit


def test_host_register_rejects_null(lib):
    assert lib.psops_host_register(None, 16) == binding.PSOPS_EINVAL
    assert lib.psops_host_register(0x10000, 0) == binding.PSOPS_EINVAL
    assert lib.psops_host_unregister(None) == binding.PSOPS_EINVAL


def test_strerror_is_distinct_per_code(lib):
    texts = {lib.psops_strerror(c).decode() for c in range(0, -9, -1)}
    assert len(texts) == 9
    assert lib.psops_strerror(-99).decode() == "unknown error code"


def test_inertia_matches_oracle_schedule(lib):
    cfg = binding.make_config(4, 100, m_max=0.9, m_min=0.3, t_max=5860, c1=0.2, c2=0.9, seed=1)
    for t in [0, 1, 10, 2930, 5859, 5860, 9999]:
        got = np.float32(binding.psops_inertia(cfg, t))
        assert got == oracle.inertia(0.9, 0.3, t, 5860)
    const = binding.make_config(4, 100, m_max=0.7, m_min=0.7, t_max=1, c1=1.5, c2=1.5, seed=1)
    assert np.float32(binding.psops_inertia(const, 0)) == np.float32(0.7)


def test_missing_library_is_an_error_not_a_fallback(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIBRARY", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        binding.load()


# ---------------------------------------------------------------------------
# Workload generators
# ---------------------------------------------------------------------------
def test_workload_shapes_follow_the_recipes():
    c = workloads.CONFIGS
    assert [(c[n].K, c[n].N) for n in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5")] == [
        (4, 61_706), (8, 1_250_000), (16, 11_173_962), (32, 25_557_032), (8, 50_000_000)]
    assert c["cfg1"].ld == 62_464 and c["cfg3"].ld == 11_174_912 and c["cfg4"].ld == 25_558_016
    assert all(c[n].ld % 1024 == 0 and 0 <= c[n].ld - c[n].N < 1024 for n in c)
    w = c["cfg2"].scaled(N=10_001)
    x, v, p = workloads.state(w)
    assert x.shape == (8, 10_240) and x.dtype == np.float32
    assert np.array_equal(p, x) and not x[:, 10_001:].any()
    assert abs(float(x[:, :10_001].std()) - 0.02) < 1e-3 and abs(float(v[:, :10_001].std()) - 1e-3) < 1e-4
    x2, _, _ = workloads.state(w)
    assert np.array_equal(x, x2)                                   # seeded
    assert np.array_equal(workloads.x_row(w, 3), x[3, :10_001])    # rows are independent streams
    assert not workloads.state(c["cfg1"].scaled(N=100))[1].any()   # v = 0 recipes


def test_loss_tables_ranges_and_deliberate_ties():
    w = workloads.CONFIGS["cfg3"]
    tab = workloads.losses(w)
    assert tab.shape == (100, 16) and tab.dtype == np.float32
    assert tab.min() >= 0.2 and tab.max() <= 2.3
    tied_lower = tied_higher = repeats = 0
    seen = np.full(16, np.inf, np.float32)
    for s in range(100):
        row = tab[s]
        where = np.flatnonzero(row == row.min())
        if where.size > 1:
            tied_higher += 1
        repeats += int(np.any(row == seen))
        seen = np.minimum(seen, row)
    assert tied_higher > 20 and repeats > 5
    # ties put the duplicate both below and above the first minimum's index over the run
    first = [int(np.argmin(r)) for r in tab]
    last = [int(16 - 1 - np.argmin(r[::-1])) for r in tab]
    assert any(a != b for a, b in zip(first, last))
    assert np.array_equal(tab, workloads.losses(w))
    plain = workloads.losses(workloads.CONFIGS["cfg4"])
    assert plain.shape == (100, 32) and plain.min() >= 0.1 and plain.max() <= 2.5


def test_sample_columns_cover_head_and_tail():
    cols = workloads.sample_columns(1000, 50, 3)
    assert cols[0] == 0 and cols[-1] == 999 and np.all(np.diff(cols) > 0)
    assert {0, 1, 2, 3, 996, 997, 998, 999} <= set(cols.tolist())


def test_bench_parity_metric_and_timing_stats():
    """The benchmark's own checker: the error measure of its `parity` object and
    the per-step statistics (host arithmetic only)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    want = np.array([[1.0, 2.0, 0.0, np.nan, np.inf, 4.0]], np.float32)
    got = want.copy()
    got[0, 2] = -0.0                                   # +0 / -0 and NaN / NaN count as identical
    assert bench._rel_err(got, want) == (0.0, 0, 0)
    got[0, 1] = np.nextafter(np.float32(2.0), np.float32(3.0))      # one ulp: inside 1e-6, not identical
    err, outside, inexact = bench._rel_err(got, want)
    assert 0 < err < 1e-6 and outside == 0 and inexact == 1
    got[0, 5] = 4.001
    got[0, 0] = np.nan                                 # a NaN on one side only is a mismatch
    err, outside, inexact = bench._rel_err(got, want)
    assert err == np.inf and outside == 2 and inexact == 3
    t = bench.Timing(0.010, [1.0, 3.0, 2.0, 4.0])
    t.window_ms_per_step = [2.0, 3.0]
    st = t.stats(4)
    assert st["ms_per_step_mean"] == 2.5 and st["per_step_ms"] == {"median": 2.5, "min": 1.0, "max": 4.0, "n": 4}
    assert st["window_ms_per_step"] == {"median": 2.5, "min": 2.0, "max": 3.0, "n": 3}
    # algorithmic bytes of a sync: 20 B per particle-element + the gBest row
    from paper_2009_03816_b200 import workloads
    w = workloads.CONFIGS["cfg4"]
    assert bench.sync_bytes(w) == 20 * 32 * 25_557_032 + 4 * 25_557_032 == 16_458_728_608
