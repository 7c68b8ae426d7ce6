"""Thin ctypes binding of ``libpsops.so`` -- argument marshalling only.

Every function has the name and meaning of the C entry point declared in
``include/psops.h``; every step of the synchronisation runs in the CUDA
library.  PyTorch is used for device memory and streams, nothing else.  If the
shared library is missing the import of a symbol fails with an error: there is
no CPU path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from .build import LIBRARY

PSOPS_OK = 0
PSOPS_EINVAL, PSOPS_EALIGN, PSOPS_ESTATE, PSOPS_ENAN = -1, -2, -3, -4
PSOPS_EWORKSPACE, PSOPS_ECUDA, PSOPS_ENOMEM, PSOPS_ELIMIT = -5, -6, -7, -8
PSOPS_STATIC_SCRATCH_DOUBLES = 1 << 20
PSOPS_MAX_K = 1024
PSOPS_KEEP_GBEST, PSOPS_QUADRATIC, PSOPS_GBEST_HISTORY, PSOPS_SEPARATE_SELECT = 1, 2, 4, 8
PSOPS_X, PSOPS_V, PSOPS_PBEST, PSOPS_GBEST = 0, 1, 2, 3

EXPORTS = [
    "psops_workspace_bytes", "psops_create", "psops_set_losses", "psops_sync",
    "psops_sync_host", "psops_average", "psops_get_weights", "psops_set_weights",
    "psops_sync_info", "psops_get_losses", "psops_set_quadratic",
    "psops_eval_quadratic", "psops_get_state", "psops_set_state", "psops_inertia",
    "psops_launch_count", "psops_strerror", "psops_last_error", "psops_destroy",
    "psops_quadratic_fitness_static", "psops_shard_select", "psops_shard_update",
    "psops_shard_update_range", "psops_get_history", "psops_set_history", "psops_ssgd",
    "psops_host_register", "psops_host_unregister",
]


class psops_config(ctypes.Structure):
    _fields_ = [("K", ctypes.c_int32), ("k_first", ctypes.c_int32), ("N", ctypes.c_int64),
                ("ld", ctypes.c_int64), ("m_max", ctypes.c_float), ("m_min", ctypes.c_float),
                ("t_max", ctypes.c_int64), ("c1", ctypes.c_float), ("c2", ctypes.c_float),
                ("seed", ctypes.c_uint64), ("flags", ctypes.c_uint32), ("K_total", ctypes.c_int32)]


class PsopsError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = f"{where}: {_strerror(code)} ({code})"
        if detail:
            msg += f": {detail}"
        super().__init__(msg)


_lib = None
_vp, _f32p, _u32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p


def load() -> ctypes.CDLL:
    """Load the CUDA library; raise if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIBRARY):
        raise ImportError(
            f"{LIBRARY} is missing: build it with "
            "`python -m paper_2009_03816_b200.build` (needs nvcc). "
            "There is no CPU fallback.")
    lib = ctypes.CDLL(LIBRARY)
    cfgp = ctypes.POINTER(psops_config)
    sig = {
        "psops_workspace_bytes": (ctypes.c_size_t, [cfgp]),
        "psops_create": (ctypes.c_int, [ctypes.POINTER(_vp), cfgp, _f32p, _f32p, _f32p, _vp,
                                        ctypes.c_size_t, _vp]),
        "psops_set_losses": (ctypes.c_int, [_vp, _f32p, ctypes.c_int]),
        "psops_sync": (ctypes.c_int, [_vp, ctypes.c_int64, ctypes.c_float]),
        "psops_sync_host": (ctypes.c_int, [_vp, _f32p, ctypes.c_int64, _f32p, ctypes.c_int64,
                                           ctypes.c_float, _f32p, ctypes.c_int64]),
        "psops_average": (ctypes.c_int, [_vp]),
        "psops_get_weights": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int, _f32p, ctypes.c_int]),
        "psops_set_weights": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int, _f32p, ctypes.c_int]),
        "psops_sync_info": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_int), _u32p, _f32p]),
        "psops_get_losses": (ctypes.c_int, [_vp, _f32p, ctypes.c_int]),
        "psops_set_quadratic": (ctypes.c_int, [_vp, _f32p, _f32p]),
        "psops_eval_quadratic": (ctypes.c_int, [_vp]),
        "psops_get_state": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_uint32), _f32p]),
        "psops_set_state": (ctypes.c_int, [_vp, ctypes.c_uint32, _f32p]),
        "psops_inertia": (ctypes.c_float, [cfgp, ctypes.c_int64]),
        "psops_launch_count": (ctypes.c_int64, [_vp]),
        "psops_strerror": (ctypes.c_char_p, [ctypes.c_int]),
        "psops_last_error": (ctypes.c_char_p, [_vp]),
        "psops_destroy": (ctypes.c_int, [_vp]),
        "psops_shard_select": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_int)]),
        "psops_shard_update": (ctypes.c_int, [_vp, ctypes.c_int64, ctypes.c_float, _f32p]),
        "psops_shard_update_range": (ctypes.c_int, [_vp, ctypes.c_int64, ctypes.c_float, _f32p,
                                                    ctypes.c_int64, ctypes.c_int64]),
        "psops_get_history": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]),
        "psops_set_history": (ctypes.c_int, [_vp, ctypes.c_float, _f32p, ctypes.c_int]),
        "psops_ssgd": (ctypes.c_int, [_vp, _f32p, ctypes.c_int64, ctypes.c_float]),
        "psops_host_register": (ctypes.c_int, [_vp, ctypes.c_size_t]),
        "psops_host_unregister": (ctypes.c_int, [_vp]),
        "psops_quadratic_fitness_static": (ctypes.c_int, [_f32p, ctypes.c_int64, ctypes.c_int32,
                                                          ctypes.c_int64, _f32p, _f32p, _f32p, _vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)            # AttributeError if a symbol is missing
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _strerror(code: int) -> str:
    try:
        return load().psops_strerror(int(code)).decode()
    except Exception:  # pragma: no cover
        return "error"


def _check(rc: int, where: str, ctx=None) -> None:
    if rc != PSOPS_OK:
        detail = ""
        if ctx is not None and rc == PSOPS_ECUDA:
            detail = load().psops_last_error(ctx).decode()
        raise PsopsError(rc, where, detail)


def _ptr(buf) -> int:
    """Address of a torch tensor or numpy array (0 for None)."""
    if buf is None:
        return 0
    if isinstance(buf, torch.Tensor):
        return buf.data_ptr()
    if isinstance(buf, np.ndarray):
        return buf.ctypes.data
    if isinstance(buf, int):
        return buf
    raise TypeError(f"cannot take the address of {type(buf)!r}")


def _on_device(buf) -> int:
    return int(isinstance(buf, torch.Tensor) and buf.is_cuda)


def make_config(K, N, ld=None, *, m_max, m_min, t_max=1, c1, c2, seed, flags=0,
                k_first=0, K_total=0) -> psops_config:
    ld = (int(N) + 3) // 4 * 4 if ld is None else int(ld)
    return psops_config(int(K), int(k_first), int(N), ld, float(m_max), float(m_min), int(t_max),
                        float(c1), float(c2), int(seed), int(flags), int(K_total))


# ---- one function per C entry point --------------------------------------

def psops_workspace_bytes(cfg: psops_config) -> int:
    return int(load().psops_workspace_bytes(ctypes.byref(cfg)))


def psops_inertia(cfg: psops_config, t_iter: int) -> float:
    return float(load().psops_inertia(ctypes.byref(cfg), int(t_iter)))


def psops_create(cfg, d_x, d_v, d_pbest, d_workspace, workspace_bytes=None, stream=None):
    handle = _vp()
    if workspace_bytes is None:
        workspace_bytes = d_workspace.numel() * d_workspace.element_size() if d_workspace is not None else 0
    rc = load().psops_create(ctypes.byref(handle), ctypes.byref(cfg), _ptr(d_x), _ptr(d_v),
                             _ptr(d_pbest), _ptr(d_workspace), int(workspace_bytes),
                             int(stream) if stream else None)
    _check(rc, "psops_create")
    return handle


def psops_set_losses(ctx, losses) -> None:
    _check(load().psops_set_losses(ctx, _ptr(losses), _on_device(losses)), "psops_set_losses", ctx)


def psops_sync(ctx, t_iter: int = 0, lam: float = 1.0) -> None:
    _check(load().psops_sync(ctx, int(t_iter), float(lam)), "psops_sync", ctx)


def psops_sync_host(ctx, h_x_in, h_in_ld, h_losses, t_iter, lam, h_x_out, h_out_ld) -> None:
    _check(load().psops_sync_host(ctx, _ptr(h_x_in), int(h_in_ld), _ptr(h_losses), int(t_iter),
                                  float(lam), _ptr(h_x_out), int(h_out_ld)), "psops_sync_host", ctx)


def psops_shard_select(ctx) -> int:
    g = ctypes.c_int(-1)
    _check(load().psops_shard_select(ctx, ctypes.byref(g)), "psops_shard_select", ctx)
    return int(g.value)


def psops_shard_update(ctx, t_iter, lam, d_gbest_row) -> None:
    _check(load().psops_shard_update(ctx, int(t_iter), float(lam), _ptr(d_gbest_row)),
           "psops_shard_update", ctx)


def psops_shard_update_range(ctx, t_iter, lam, d_gbest_row, first_elem, last_elem) -> None:
    _check(load().psops_shard_update_range(ctx, int(t_iter), float(lam), _ptr(d_gbest_row),
                                           int(first_elem), int(last_elem)),
           "psops_shard_update_range", ctx)


def psops_get_history(ctx):
    loss, valid = ctypes.c_float(0.0), ctypes.c_int(0)
    _check(load().psops_get_history(ctx, ctypes.byref(loss), ctypes.byref(valid)), "psops_get_history", ctx)
    return float(loss.value), bool(valid.value)


def psops_set_history(ctx, gbest_loss, gbest_row) -> None:
    _check(load().psops_set_history(ctx, float(gbest_loss), _ptr(gbest_row), _on_device(gbest_row)),
           "psops_set_history", ctx)


def psops_ssgd(ctx, d_grad, grad_ld, alpha) -> None:
    _check(load().psops_ssgd(ctx, _ptr(d_grad), int(grad_ld), float(alpha)), "psops_ssgd", ctx)


def psops_host_register(buf) -> None:
    """Pin a host buffer (numpy array or CPU tensor) in place for psops_sync_host."""
    nbytes = buf.nbytes if isinstance(buf, np.ndarray) else buf.numel() * buf.element_size()
    _check(load().psops_host_register(_ptr(buf), int(nbytes)), "psops_host_register")


def psops_host_unregister(buf) -> None:
    _check(load().psops_host_unregister(_ptr(buf)), "psops_host_unregister")


def psops_average(ctx) -> None:
    _check(load().psops_average(ctx), "psops_average", ctx)


def psops_get_weights(ctx, which: int, k: int, dst) -> None:
    _check(load().psops_get_weights(ctx, int(which), int(k), _ptr(dst), _on_device(dst)),
           "psops_get_weights", ctx)


def psops_set_weights(ctx, which: int, k: int, src) -> None:
    _check(load().psops_set_weights(ctx, int(which), int(k), _ptr(src), _on_device(src)),
           "psops_set_weights", ctx)


def psops_sync_info(ctx, K: int):
    g = ctypes.c_int(-1)
    words = np.zeros((K + 31) // 32, dtype=np.uint32)
    pl = np.zeros(K, dtype=np.float32)
    _check(load().psops_sync_info(ctx, ctypes.byref(g), _ptr(words), _ptr(pl)), "psops_sync_info", ctx)
    improved = np.array([(int(words[i >> 5]) >> (i & 31)) & 1 for i in range(K)], dtype=bool)
    return int(g.value), improved, pl


def psops_get_losses(ctx, dst) -> None:
    _check(load().psops_get_losses(ctx, _ptr(dst), _on_device(dst)), "psops_get_losses", ctx)


def psops_set_quadratic(ctx, d_dvec, d_tvec) -> None:
    _check(load().psops_set_quadratic(ctx, _ptr(d_dvec), _ptr(d_tvec)), "psops_set_quadratic", ctx)


def psops_eval_quadratic(ctx) -> None:
    _check(load().psops_eval_quadratic(ctx), "psops_eval_quadratic", ctx)


def psops_get_state(ctx, K: int):
    step = ctypes.c_uint32(0)
    pl = np.zeros(K, dtype=np.float32)
    _check(load().psops_get_state(ctx, ctypes.byref(step), _ptr(pl)), "psops_get_state", ctx)
    return int(step.value), pl


def psops_set_state(ctx, sync_step: int, pbest_loss) -> None:
    pl = np.ascontiguousarray(pbest_loss, dtype=np.float32)
    _check(load().psops_set_state(ctx, int(sync_step), _ptr(pl)), "psops_set_state", ctx)


def psops_launch_count(ctx) -> int:
    return int(load().psops_launch_count(ctx))


def psops_destroy(ctx) -> None:
    _check(load().psops_destroy(ctx), "psops_destroy")


def psops_quadratic_fitness_static(d_x, ld, K, N, d_dvec, d_tvec, d_loss, stream=None) -> None:
    """Fitness of K device rows into d_loss[K] using the library's built-in
    scratch array: no workspace, no context, no allocation (for callers that
    cannot allocate device memory).  Work is enqueued on `stream`."""
    _check(load().psops_quadratic_fitness_static(_ptr(d_x), int(ld), int(K), int(N), _ptr(d_dvec),
                                                 _ptr(d_tvec), _ptr(d_loss),
                                                 int(stream) if stream else None),
           "psops_quadratic_fitness_static")


# ---- convenience holder of the tensors a context borrows ------------------

class Swarm:
    """Owns the device tensors (torch) that one psops context borrows and
    forwards to the C entry points.  No arithmetic happens here."""

    def __init__(self, x, v, pbest, *, N=None, m_max, m_min, t_max=1, c1, c2, seed, flags=0,
                 stream=None, k_first=0, K_total=0):
        for t in (x, v, pbest):
            assert t.is_cuda and t.dtype == torch.float32 and t.dim() == 2 and t.stride(1) == 1
        self.x, self.v, self.pbest = x, v, pbest
        self.K = x.shape[0]
        self.ld = x.stride(0)
        assert v.stride(0) == self.ld and pbest.stride(0) == self.ld
        self.N = int(N) if N is not None else x.shape[1]
        self.cfg = make_config(self.K, self.N, self.ld, m_max=m_max, m_min=m_min, t_max=t_max,
                               c1=c1, c2=c2, seed=seed, flags=flags, k_first=k_first, K_total=K_total)
        self.Kt = K_total if K_total else self.K
        nbytes = psops_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise PsopsError(PSOPS_EINVAL, "psops_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=x.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(x.device).cuda_stream
        self._refs = []
        self.ctx = psops_create(self.cfg, x, v, pbest, self.workspace, nbytes, self.stream)

    def set_losses(self, losses):
        if isinstance(losses, (list, tuple)):
            losses = np.asarray(losses, dtype=np.float32)
        if isinstance(losses, np.ndarray):
            losses = np.ascontiguousarray(losses, dtype=np.float32)
        count = losses.size if isinstance(losses, np.ndarray) else losses.numel()
        assert count == self.Kt
        self._loss_ref = losses        # a device buffer is read by the next sync: keep it alive
        psops_set_losses(self.ctx, losses)

    def sync(self, t_iter=0, lam=1.0):
        psops_sync(self.ctx, t_iter, lam)

    def sync_host(self, h_x_in, h_losses, t_iter=0, lam=1.0, h_x_out=None):
        h_x_out = h_x_in if h_x_out is None else h_x_out
        h_losses = np.ascontiguousarray(h_losses, dtype=np.float32) \
            if not isinstance(h_losses, torch.Tensor) else h_losses
        psops_sync_host(self.ctx, h_x_in, _ld_of(h_x_in), h_losses, t_iter, lam, h_x_out, _ld_of(h_x_out))

    def average(self):
        psops_average(self.ctx)

    def info(self):
        return psops_sync_info(self.ctx, self.Kt)

    def shard_select(self) -> int:
        return psops_shard_select(self.ctx)

    def shard_update(self, d_gbest_row, t_iter=0, lam=1.0):
        psops_shard_update(self.ctx, t_iter, lam, d_gbest_row)

    def shard_update_range(self, d_gbest_row, first_elem, last_elem, t_iter=0, lam=1.0):
        psops_shard_update_range(self.ctx, t_iter, lam, d_gbest_row, first_elem, last_elem)

    def ssgd(self, d_grad, alpha):
        psops_ssgd(self.ctx, d_grad, d_grad.stride(0), alpha)

    def history(self):
        return psops_get_history(self.ctx)

    def losses(self) -> np.ndarray:
        out = np.zeros(self.Kt, dtype=np.float32)
        psops_get_losses(self.ctx, out)
        return out

    def row(self, which, k=0) -> np.ndarray:
        out = np.empty(self.N, dtype=np.float32)
        psops_get_weights(self.ctx, which, k, out)
        return out

    def set_quadratic(self, dvec, tvec):
        self._refs = [dvec, tvec]
        psops_set_quadratic(self.ctx, dvec, tvec)

    def eval_quadratic(self):
        psops_eval_quadratic(self.ctx)

    def state(self):
        return psops_get_state(self.ctx, self.Kt)

    def set_state(self, step, pbest_loss):
        psops_set_state(self.ctx, step, pbest_loss)

    @property
    def launches(self) -> int:
        return psops_launch_count(self.ctx)

    def close(self):
        if self.ctx is not None:
            psops_destroy(self.ctx)
            self.ctx = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


def _ld_of(buf) -> int:
    if isinstance(buf, torch.Tensor):
        return buf.stride(0)
    return buf.strides[0] // buf.itemsize
