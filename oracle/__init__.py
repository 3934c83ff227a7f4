"""ctypes front end of the DaSGD CPU oracle -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It compiles ``dasgd_oracle.cpp`` with g++ (twice: a single-thread build
and an OpenMP build of the same source) and exposes the C functions through a
small numpy-facing class.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dasgd_oracle.cpp")
_HDR = os.path.join(_HERE, "dasgd_oracle.h")
_LIBS = {False: os.path.join(_HERE, "liboracle_dasgd.so"),
         True: os.path.join(_HERE, "liboracle_dasgd_omp.so")}

F32, BF16_MASTER_F32 = 0, 1
MERGE_XI, MERGE_DELTA = 0, 1


def build(force: bool = False) -> None:
    """Compile both builds of the oracle if missing or older than the source."""
    for omp, lib in _LIBS.items():
        if (not force and os.path.exists(lib)
                and os.path.getmtime(lib) >= max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))):
            continue
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-ffp-contract=off", _SRC, "-o", lib + ".tmp"]
        if omp:
            cmd.insert(1, "-fopenmp")
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(lib + ".tmp", lib)


_loaded: dict[bool, ctypes.CDLL] = {}


def bind(path: str) -> ctypes.CDLL:
    """Load one build of the oracle and declare its signatures."""
    L = ctypes.CDLL(path)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    L.oracle_dasgd_create.restype = vp
    L.oracle_dasgd_create.argtypes = [i32, i64, i32, i32, f32, f32, f32, i32, i32]
    L.oracle_dasgd_destroy.restype = None
    L.oracle_dasgd_destroy.argtypes = [vp]
    L.oracle_dasgd_set_state.argtypes = [vp, vp, vp]
    L.oracle_dasgd_get_state.argtypes = [vp, vp, vp, vp]
    L.oracle_dasgd_steps_done.restype = i64
    L.oracle_dasgd_steps_done.argtypes = [vp]
    L.oracle_dasgd_pending.argtypes = [vp]
    L.oracle_dasgd_get_pending.argtypes = [vp, i32, ctypes.POINTER(i64), vp, vp]
    L.oracle_dasgd_local_step.argtypes = [vp, vp, f32]
    L.oracle_dasgd_snapshot.argtypes = [vp]
    L.oracle_dasgd_average.argtypes = [vp]
    L.oracle_dasgd_merge.argtypes = [vp]
    L.oracle_dasgd_step.argtypes = [vp, vp, f32]
    L.oracle_dasgd_set_variant.argtypes = [vp, i32, i32]
    L.oracle_dasgd_set_momentum_averaging.argtypes = [vp, i32]
    L.oracle_dasgd_get_pending_momentum.argtypes = [vp, i32, vp, vp]
    L.oracle_dasgd_set_shard.argtypes = [vp, i32]
    L.oracle_dasgd_partial_sum.argtypes = [vp, vp]
    L.oracle_dasgd_set_mean_from_sum.argtypes = [vp, vp]
    L.oracle_dasgd_threads.argtypes = []
    f64, pi32 = ctypes.c_double, ctypes.POINTER(i32)
    L.oracle_dasgd_delay_guideline.argtypes = [f64, f64, pi32, pi32]
    L.oracle_dasgd_delay_from_system.argtypes = [f64, f64, f64, f64, f64, f64, pi32, pi32]
    return L


def _lib(omp: bool) -> ctypes.CDLL:
    if omp not in _loaded:
        build()
        _loaded[omp] = bind(_LIBS[omp])
    return _loaded[omp]


class OracleError(RuntimeError):
    pass


def delay_guideline(t_c: float, t_p: float):
    """(d, tau) of the paper's guideline: smallest d with t_c < d*t_p; tau = d + 1."""
    d, tau = ctypes.c_int32(), ctypes.c_int32()
    if _lib(False).oracle_dasgd_delay_guideline(t_c, t_p, ctypes.byref(d), ctypes.byref(tau)) != 0:
        raise OracleError("delay_guideline: need t_c >= 0 and t_p > 0")
    return d.value, tau.value


def delay_from_system(m, n_p, BW, B_l, FLOP, FLOPS):
    d, tau = ctypes.c_int32(), ctypes.c_int32()
    if _lib(False).oracle_dasgd_delay_from_system(m, n_p, BW, B_l, FLOP, FLOPS, ctypes.byref(d), ctypes.byref(tau)) != 0:
        raise OracleError("delay_from_system: bad arguments")
    return d.value, tau.value


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


class OracleDaSGD:
    """K replicas of a P-vector driven by the oracle.  Arrays are numpy, [K][P]."""

    def __init__(self, K, P, tau, d, xi, momentum=0.0, weight_decay=0.0, dtype=F32,
                 merge_mode=MERGE_XI, omp=False, nesterov=False, decoupled_wd=False, average_momentum=False):
        self._L = _lib(omp)
        self.K, self.P, self.tau, self.d, self.dtype = K, P, tau, d, dtype
        self._h = self._L.oracle_dasgd_create(K, P, tau, d, xi, momentum, weight_decay, dtype, merge_mode)
        if not self._h:
            raise OracleError("invalid configuration")
        if (nesterov or decoupled_wd) and self._L.oracle_dasgd_set_variant(self._h, int(nesterov), int(decoupled_wd)) != 0:
            raise OracleError("invalid variant (Nesterov needs momentum)")
        if average_momentum and self._L.oracle_dasgd_set_momentum_averaging(self._h, 1) != 0:
            raise OracleError("momentum averaging needs momentum > 0")

    def close(self):
        if getattr(self, "_h", None):
            self._L.oracle_dasgd_destroy(self._h)
            self._h = None

    __del__ = close

    def _chk(self, rc, what):
        if rc != 0:
            raise OracleError(f"{what} failed with code {rc}")

    def _grad(self, g):
        g = np.ascontiguousarray(g)
        want = np.float32 if self.dtype == F32 else np.uint16
        if g.dtype != want or g.shape != (self.K, self.P):
            raise OracleError(f"gradients must be {want.__name__} [{self.K}][{self.P}]")
        return g

    @property
    def threads(self):
        return self._L.oracle_dasgd_threads()

    def set_state(self, w, m=None):
        w = np.ascontiguousarray(w, dtype=np.float32)
        if w.ndim == 1:  # shared start
            w = np.ascontiguousarray(np.broadcast_to(w, (self.K, self.P)))
        assert w.shape == (self.K, self.P)
        if m is not None:
            m = np.ascontiguousarray(m, dtype=np.float32)
            assert m.shape == (self.K, self.P)
        self._chk(self._L.oracle_dasgd_set_state(self._h, _ptr(w), _ptr(m)), "set_state")

    @property
    def w(self):
        out = np.empty((self.K, self.P), np.float32)
        self._chk(self._L.oracle_dasgd_get_state(self._h, _ptr(out), None, None), "get_state")
        return out

    @property
    def m(self):
        out = np.empty((self.K, self.P), np.float32)
        self._chk(self._L.oracle_dasgd_get_state(self._h, None, _ptr(out), None), "get_state")
        return out

    @property
    def w_lp(self):
        out = np.empty((self.K, self.P), np.uint16)
        self._chk(self._L.oracle_dasgd_get_state(self._h, None, None, _ptr(out)), "get_state")
        return out

    @property
    def t(self):
        return self._L.oracle_dasgd_steps_done(self._h)

    @property
    def n_pending(self):
        return self._L.oracle_dasgd_pending(self._h)

    def pending(self, i=0, want_snap=True, want_mean=True):
        s = ctypes.c_int64()
        snap = np.empty((self.K, self.P), np.float32) if want_snap else None
        mean = np.empty((self.P,), np.float32) if want_mean else None
        self._chk(self._L.oracle_dasgd_get_pending(self._h, i, ctypes.byref(s), _ptr(snap), _ptr(mean)),
                  "get_pending")
        return s.value, snap, mean

    def pending_momentum(self, i=0, want_mean=True):
        snap = np.empty((self.K, self.P), np.float32)
        mean = np.empty((self.P,), np.float32) if want_mean else None
        self._chk(self._L.oracle_dasgd_get_pending_momentum(self._h, i, _ptr(snap), _ptr(mean)), "get_pending_momentum")
        return snap, mean

    def local_step(self, g, lr):
        self._chk(self._L.oracle_dasgd_local_step(self._h, _ptr(self._grad(g)), lr), "local_step")

    def snapshot(self):
        self._chk(self._L.oracle_dasgd_snapshot(self._h), "snapshot")

    def average(self):
        self._chk(self._L.oracle_dasgd_average(self._h), "average")

    def merge(self):
        self._chk(self._L.oracle_dasgd_merge(self._h), "merge")

    def step(self, g, lr):
        self._chk(self._L.oracle_dasgd_step(self._h, _ptr(self._grad(g)), lr), "step")

    # -- a shard of the worker axis -----------------------------------------
    def set_shard(self, K_total):
        """This object holds K of K_total workers; the mean then needs the partial sums of all shards."""
        self._chk(self._L.oracle_dasgd_set_shard(self._h, K_total), "set_shard")
        self.K_total = K_total

    def partial_sum(self):
        """float64 [P]: sum over this shard's workers of the oldest snapshot without a mean."""
        out = np.empty((self.P,), np.float64)
        self._chk(self._L.oracle_dasgd_partial_sum(self._h, _ptr(out)), "partial_sum")
        return out

    def set_mean_from_sum(self, total):
        total = np.ascontiguousarray(total, dtype=np.float64)
        assert total.shape == (self.P,)
        self._chk(self._L.oracle_dasgd_set_mean_from_sum(self._h, _ptr(total)), "set_mean_from_sum")

    def sharded_step(self, g, lr, exchange):
        """One iteration of the schedule on a shard: `exchange(partial_sum) -> total` is the all-reduce."""
        self.local_step(g, lr)
        u = self.t
        if self.d > 0 and u - self.d >= self.tau and (u - self.d) % self.tau == 0:
            self.merge()
        if u % self.tau == 0:
            self.snapshot()
            self.set_mean_from_sum(exchange(self.partial_sum()))
            if self.d == 0:
                self.merge()
