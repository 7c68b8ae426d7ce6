"""Helpers shared by the GPU parity tests: device buffers with guard bands,
the tolerance of the parity contract, and a lock-step driver that feeds the
same seeded inputs to the CUDA library and to the CPU oracle."""
import os

import numpy as np
import torch

import oracle
from paper_2009_03816_b200 import binding
from paper_2009_03816_b200 import build as _build

NTHREADS = max(1, os.cpu_count() or 1)
GUARD = 64                       # floats of canary before and after each buffer
CANARY = np.float32(-7.25e33)


def ensure_library():
    _build.build_library()
    return binding.load()


def assert_close(got, want, what=""):
    """The parity contract: |gpu - ref| <= 1e-6 * max(|ref|, eps) element-wise,
    eps = 1e-6 * RMS(ref).  Returns the number of elements that are not
    bit-identical (expected 0: both sides use the same rounding sequence)."""
    got = np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if got.dtype == np.float32 and want.dtype == np.float32 and got.flags.c_contiguous and want.flags.c_contiguous \
            and np.array_equal(got.view(np.uint32), want.view(np.uint32)):
        return 0                                          # identical bits: nothing more to look at
    rms = float(np.sqrt(np.mean(want.astype(np.float64) ** 2))) if want.size else 0.0
    tol = 1e-6 * np.maximum(np.abs(want).astype(np.float64), 1e-6 * rms)
    diff = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bad = ~(diff <= tol)                                  # NaN counts as bad ...
    bad &= ~((got == want) | (np.isnan(got) & np.isnan(want)))   # ... unless both agree
    if bad.any():
        idx = np.argwhere(bad)[0]
        raise AssertionError(
            f"{what}: {int(bad.sum())} of {got.size} outside 1e-6; first at {tuple(idx)}: "
            f"gpu={got[tuple(idx)]!r} ref={want[tuple(idx)]!r}")
    same = (got.view(np.uint32) == want.view(np.uint32)) | ((got == 0) & (want == 0))
    return int(got.size - same.sum())


def device_compare(dev_rows, want, what="", rows_per_piece=4):
    """The same contract for a whole swarm without bringing it to the host: the
    oracle's rows are uploaded piece by piece and compared on the device (plain
    torch comparisons; this is the checker, not the path).  Returns the number of
    elements that are not bit-identical (+0 and -0 count as identical); raises if
    any element is outside |gpu - ref| <= 1e-6 * max(|ref|, 1e-6 * RMS(ref))."""
    K, n = want.shape
    assert tuple(dev_rows.shape) == (K, n), (what, tuple(dev_rows.shape), want.shape)
    rms = float(np.sqrt(np.mean(np.square(want, dtype=np.float64))))
    inexact = 0
    for k0 in range(0, K, rows_per_piece):
        ref = torch.from_numpy(np.ascontiguousarray(want[k0:k0 + rows_per_piece])).to(dev_rows.device)
        got = dev_rows[k0:k0 + rows_per_piece]
        differ = (got.view(torch.int32) != ref.view(torch.int32)) & ~((got == 0) & (ref == 0))
        n_differ = int(differ.sum().item())
        if n_differ:
            tol = 1e-6 * torch.clamp(ref.abs().double(), min=1e-6 * rms)
            outside = ~((got.double() - ref.double()).abs() <= tol) & differ
            n_out = int(outside.sum().item())
            if n_out:
                idx = torch.nonzero(outside)[0].tolist()
                raise AssertionError(
                    f"{what}: {n_out} elements of rows {k0}.. outside 1e-6; first at "
                    f"({k0 + idx[0]}, {idx[1]}): gpu={got[idx[0], idx[1]].item()!r} ref={ref[idx[0], idx[1]].item()!r}")
        inexact += n_differ
        del ref, differ
    return inexact


class DeviceRows:
    """K rows of stride ld inside a larger CUDA buffer with canaries before the
    first row, after the last row and in the padding [N, ld) of every row.
    ``offset`` shifts the first row by that many floats to break 16-byte
    alignment."""

    def __init__(self, host_rows, N, ld, offset=0, device="cuda:0"):
        K = host_rows.shape[0]
        self.K, self.N, self.ld, self.offset = K, N, ld, offset
        total = GUARD + offset + K * ld + GUARD
        buf = np.full(total, CANARY, dtype=np.float32)
        body = buf[GUARD + offset: GUARD + offset + K * ld].reshape(K, ld)
        body[:, :N] = host_rows[:, :N]
        self.raw = torch.from_numpy(buf).to(device)
        self.rows = self.raw[GUARD + offset: GUARD + offset + K * ld].view(K, ld)

    def host(self):
        return self.rows.cpu().numpy()[:, :self.N]

    def check_canaries(self, what=""):
        buf = self.raw.cpu().numpy()
        lo = GUARD + self.offset
        assert np.all(buf[:lo] == CANARY), f"{what}: wrote before the buffer"
        assert np.all(buf[lo + self.K * self.ld:] == CANARY), f"{what}: wrote past the buffer"
        if self.ld > self.N:
            body = buf[lo: lo + self.K * self.ld].reshape(self.K, self.ld)
            assert np.all(body[:, self.N:] == CANARY), f"{what}: wrote into the row padding"


class Pair:
    """The CUDA swarm and the oracle swarm on the same initial state."""

    def __init__(self, x, v, p, N, *, ld=None, offset=0, m_max, m_min, t_max=1, c1, c2, seed,
                 flags=0, elem_index=None):
        ensure_library()
        K = x.shape[0]
        ld = (N + 3) // 4 * 4 if ld is None else ld
        self.K, self.N = K, N
        self.dx = DeviceRows(x, N, ld, offset)
        self.dv = DeviceRows(v, N, ld, offset)
        self.dp = DeviceRows(p, N, ld, offset)
        self.gpu = binding.Swarm(self.dx.rows, self.dv.rows, self.dp.rows, N=N, m_max=m_max,
                                 m_min=m_min, t_max=t_max, c1=c1, c2=c2, seed=seed, flags=flags)
        self.ref = oracle.RefSwarm(x[:, :N], v[:, :N], p[:, :N], m_max=m_max, m_min=m_min,
                                   t_max=t_max, c1=c1, c2=c2, seed=seed, nthreads=NTHREADS,
                                   elem_index=elem_index)
        self.inexact = 0

    def sync(self, loss, t=0, lam=1.0, want_gbest=False):
        loss = np.ascontiguousarray(loss, dtype=np.float32)
        self.gpu.set_losses(loss)
        self.gpu.sync(t, lam)
        self.ref.sync(loss, t, lam, want_gbest=want_gbest)

    def check_selection(self):
        g, improved, pl = self.gpu.info()
        assert g == self.ref.g, (g, self.ref.g)
        assert np.array_equal(improved, self.ref.improved)
        assert np.array_equal(pl.view(np.uint32), self.ref.pbest_loss.view(np.uint32))

    def check_state(self, what=""):
        self.inexact += assert_close(self.dx.host(), self.ref.x, what + " x")
        self.inexact += assert_close(self.dv.host(), self.ref.v, what + " v")
        self.inexact += assert_close(self.dp.host(), self.ref.p, what + " pbest")

    def check_canaries(self, what=""):
        for name, d in (("x", self.dx), ("v", self.dv), ("pbest", self.dp)):
            d.check_canaries(f"{what} {name}")

    def close(self):
        self.gpu.close()
