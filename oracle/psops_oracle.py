"""ctypes front end of the plain-C oracle in ``psops_ref.c``.

TEST INFRASTRUCTURE ONLY: the slow CPU reference that the CUDA library is
compared with.  Argument marshalling only; all arithmetic is in the C file,
which states the passage of the paper each function follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psops_ref.c")
_LIB = os.path.join(_HERE, "libpsops_ref.so")
_lock = threading.Lock()
_lib = None

# No -ffast-math, no contraction: every rounding is the one written in the C.
_CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-fPIC", "-shared", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Compile ``psops_ref.c`` with gcc into ``libpsops_ref.so`` beside it."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < os.path.getmtime(_SRC))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *_CFLAGS, _SRC, "-o", tmp, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_f32p = ctypes.POINTER(ctypes.c_float)
_u32p = ctypes.POINTER(ctypes.c_uint32)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_i64p = ctypes.POINTER(ctypes.c_int64)


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        # PSOPS_REF_LIB: the mutation tests point this at deliberately broken
        # builds of the oracle to show that the pins notice.
        lib = ctypes.CDLL(os.environ.get("PSOPS_REF_LIB") or build())
        lib.psops_ref_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
        lib.psops_ref_philox4x32_10.restype = None
        lib.psops_ref_uniform.argtypes = [ctypes.c_uint32]
        lib.psops_ref_uniform.restype = ctypes.c_float
        lib.psops_ref_draw.argtypes = [ctypes.c_uint64, ctypes.c_uint32,
                                       ctypes.c_uint32, ctypes.c_uint64,
                                       _f32p, _f32p]
        lib.psops_ref_draw.restype = None
        lib.psops_ref_inertia.argtypes = [ctypes.c_float, ctypes.c_float,
                                          ctypes.c_int64, ctypes.c_int64]
        lib.psops_ref_inertia.restype = ctypes.c_float
        lib.psops_ref_argmin.argtypes = [_f32p, ctypes.c_int]
        lib.psops_ref_argmin.restype = ctypes.c_int
        lib.psops_ref_pbest_select.argtypes = [_f32p, _f32p, ctypes.c_int, _u8p]
        lib.psops_ref_pbest_select.restype = None
        lib.psops_ref_update_element.argtypes = [ctypes.c_float] * 9 + [_f32p, _f32p]
        lib.psops_ref_update_element.restype = None
        lib.psops_ref_sync.argtypes = [
            ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _f32p, _f32p, _f32p,
            _f32p, _f32p,
            ctypes.c_float, ctypes.c_float, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_float, ctypes.c_float, ctypes.c_float,
            ctypes.c_uint64, ctypes.c_uint32,
            _i64p, _f32p, ctypes.POINTER(ctypes.c_int), _u8p, _f32p,
            _f32p, _f32p, ctypes.POINTER(ctypes.c_int),
            ctypes.c_int]
        lib.psops_ref_sync.restype = ctypes.c_int
        lib.psops_ref_average.argtypes = [ctypes.c_int, ctypes.c_int64,
                                          ctypes.c_int64, _f32p, ctypes.c_int]
        lib.psops_ref_average.restype = None
        lib.psops_ref_ssgd.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _f32p,
                                       _f32p, ctypes.c_int64, ctypes.c_float, ctypes.c_int]
        lib.psops_ref_ssgd.restype = None
        lib.psops_ref_quadratic_fitness.argtypes = [_f32p, _f32p, _f32p,
                                                    ctypes.c_int64]
        lib.psops_ref_quadratic_fitness.restype = ctypes.c_float
        lib.psops_ref_quadratic_losses.argtypes = [
            ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _f32p, _f32p, _f32p,
            _f32p, ctypes.c_int]
        lib.psops_ref_quadratic_losses.restype = None
        _lib = lib
        return lib


def _f32(a: np.ndarray):
    assert a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(_f32p)


def _rows(a: np.ndarray):
    """(K, n, ld) of a 2-D fp32 array whose rows are contiguous."""
    assert a.ndim == 2 and a.dtype == np.float32
    assert a.strides[1] == 4 and a.strides[0] % 4 == 0
    return a.shape[0], a.shape[1], a.strides[0] // 4


def philox4x32_10(ctr, key) -> np.ndarray:
    c = (ctypes.c_uint32 * 4)(*[int(w) & 0xFFFFFFFF for w in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(w) & 0xFFFFFFFF for w in key])
    o = (ctypes.c_uint32 * 4)()
    _load().psops_ref_philox4x32_10(c, k, o)
    return np.array(list(o), dtype=np.uint32)


def uniform(word: int) -> np.float32:
    return np.float32(_load().psops_ref_uniform(int(word) & 0xFFFFFFFF))


def draw(seed: int, s: int, i: int, d: int):
    r1, r2 = ctypes.c_float(), ctypes.c_float()
    _load().psops_ref_draw(int(seed), int(s), int(i), int(d),
                           ctypes.byref(r1), ctypes.byref(r2))
    return np.float32(r1.value), np.float32(r2.value)


def inertia(m_max, m_min, t, t_max) -> np.float32:
    return np.float32(_load().psops_ref_inertia(float(np.float32(m_max)),
                                                float(np.float32(m_min)),
                                                int(t), int(t_max)))


def argmin(loss) -> int:
    loss = np.ascontiguousarray(loss, dtype=np.float32)
    return int(_load().psops_ref_argmin(_f32(loss), loss.size))


def pbest_select(loss, pbest_loss):
    """Returns (improved[K] bool, new pbest_loss[K]); inputs are not modified."""
    loss = np.ascontiguousarray(loss, dtype=np.float32)
    pl = np.array(pbest_loss, dtype=np.float32, copy=True)
    imp = np.zeros(loss.size, dtype=np.uint8)
    _load().psops_ref_pbest_select(_f32(loss), _f32(pl), loss.size,
                                   imp.ctypes.data_as(_u8p))
    return imp.astype(bool), pl


def update_element(m, k1, k2, r1, r2, xo, vo, pp, gb):
    vn, xn = ctypes.c_float(), ctypes.c_float()
    args = [float(np.float32(a)) for a in (m, k1, k2, r1, r2, xo, vo, pp, gb)]
    _load().psops_ref_update_element(*args, ctypes.byref(vn), ctypes.byref(xn))
    return np.float32(vn.value), np.float32(xn.value)


def sync(x, v, p, loss, pbest_loss, *, m_max, m_min, t, t_max, c1, c2, lam,
         seed, s, elem_index=None, fixed_r=None, nthreads=1, want_gbest=False, history=None):
    """One synchronisation in place on x, v, p (2-D fp32, rows contiguous) and
    pbest_loss (1-D fp32).  Returns (g, improved[K] bool, gbest row or None).
    history: None, or a dict {"row": n fp32, "loss": 1 fp32, "valid": 1 int32}
    updated in place (gBest from the history of all particles)."""
    K, n, ld = _rows(x)
    assert _rows(v) == (K, n, ld) and _rows(p) == (K, n, ld)
    loss = np.ascontiguousarray(loss, dtype=np.float32)
    assert loss.size == K and pbest_loss.dtype == np.float32 and pbest_loss.size == K
    ei = None
    if elem_index is not None:
        elem_index = np.ascontiguousarray(elem_index, dtype=np.int64)
        assert elem_index.size == n
        ei = elem_index.ctypes.data_as(_i64p)
    fr = None
    if fixed_r is not None:
        fixed_r = np.ascontiguousarray(fixed_r, dtype=np.float32)
        assert fixed_r.size == 2
        fr = _f32(fixed_r)
    g = ctypes.c_int(-1)
    imp = np.zeros(K, dtype=np.uint8)
    gb = np.empty(n, dtype=np.float32) if want_gbest else None
    rc = _load().psops_ref_sync(
        K, n, ld, x.ctypes.data_as(_f32p), v.ctypes.data_as(_f32p),
        p.ctypes.data_as(_f32p), _f32(loss), _f32(pbest_loss),
        float(np.float32(m_max)), float(np.float32(m_min)), int(t), int(t_max),
        float(np.float32(c1)), float(np.float32(c2)), float(np.float32(lam)),
        int(seed), int(s), ei, fr, ctypes.byref(g), imp.ctypes.data_as(_u8p),
        _f32(gb) if gb is not None else None,
        _f32(history["row"]) if history else None,
        _f32(history["loss"]) if history else None,
        history["valid"].ctypes.data_as(ctypes.POINTER(ctypes.c_int)) if history else None,
        int(nthreads))
    if rc != 0:
        raise MemoryError("psops_ref_sync: allocation failed")
    return int(g.value), imp.astype(bool), gb


def average(x, nthreads=1) -> None:
    K, n, ld = _rows(x)
    _load().psops_ref_average(K, n, ld, x.ctypes.data_as(_f32p), int(nthreads))


def ssgd(w, grad, alpha, nthreads=1) -> None:
    """w (K rows) <- w[0] + (alpha / K) * sum_k grad[k], written to every row."""
    K, n, ld = _rows(w)
    Kg, ng, gld = _rows(grad)
    assert (Kg, ng) == (K, n)
    _load().psops_ref_ssgd(K, n, ld, w.ctypes.data_as(_f32p), grad.ctypes.data_as(_f32p), gld,
                           float(np.float32(alpha)), int(nthreads))


def quadratic_fitness(x, dvec, tvec) -> np.float32:
    x = np.ascontiguousarray(x, dtype=np.float32)
    dvec = np.ascontiguousarray(dvec, dtype=np.float32)
    tvec = np.ascontiguousarray(tvec, dtype=np.float32)
    assert x.ndim == 1 and dvec.shape == x.shape and tvec.shape == x.shape
    return np.float32(_load().psops_ref_quadratic_fitness(
        _f32(x), _f32(dvec), _f32(tvec), x.size))


def quadratic_losses(x, dvec, tvec, nthreads=1) -> np.ndarray:
    K, n, ld = _rows(x)
    dvec = np.ascontiguousarray(dvec, dtype=np.float32)
    tvec = np.ascontiguousarray(tvec, dtype=np.float32)
    assert dvec.size == n and tvec.size == n
    out = np.empty(K, dtype=np.float32)
    _load().psops_ref_quadratic_losses(K, n, ld, x.ctypes.data_as(_f32p),
                                       _f32(dvec), _f32(tvec), _f32(out),
                                       int(nthreads))
    return out


class RefSwarm:
    """The state one synchronisation context carries (Table I of the paper:
    positions = weights, fitness = loss, pBest memory), driven by the oracle.

    x, v, p are adopted (copied) at construction; pBest_loss starts at +inf
    (Algorithm 2 clones weights only) and the sync counter at 0.
    """

    def __init__(self, x, v, p, *, m_max, m_min, t_max, c1, c2, seed,
                 elem_index=None, nthreads=1, history=False):
        self.x = np.array(x, dtype=np.float32, copy=True, order="C")
        self.v = np.array(v, dtype=np.float32, copy=True, order="C")
        self.p = np.array(p, dtype=np.float32, copy=True, order="C")
        self.K = self.x.shape[0]
        self.pbest_loss = np.full(self.K, np.inf, dtype=np.float32)
        self.s = 0
        self.cfg = dict(m_max=m_max, m_min=m_min, t_max=t_max, c1=c1, c2=c2,
                        seed=seed)
        self.elem_index = elem_index
        self.nthreads = nthreads
        self.g = -1
        self.improved = np.zeros(self.K, dtype=bool)
        self.gbest = None
        self.history = None
        if history:
            self.history = {"row": np.zeros(self.x.shape[1], np.float32),
                            "loss": np.full(1, np.inf, np.float32),
                            "valid": np.zeros(1, np.int32)}

    def sync(self, loss, t=0, lam=1.0, want_gbest=False):
        self.g, self.improved, self.gbest = sync(
            self.x, self.v, self.p, loss, self.pbest_loss, t=t, lam=lam,
            s=self.s, elem_index=self.elem_index, nthreads=self.nthreads,
            want_gbest=want_gbest, history=self.history, **self.cfg)
        self.s += 1
        return self.g, self.improved

    def average(self):
        average(self.x, self.nthreads)
