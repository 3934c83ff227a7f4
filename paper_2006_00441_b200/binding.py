"""ctypes binding of libdasgd.so: argument marshalling only.

Every step of the path (local step, snapshot, worker-axis mean, merge, scheduling) runs inside
the native library; torch is used here for device memory and streams.  If the library cannot be
loaded the import fails -- there is no other implementation to fall back to.

The module-level ``dasgd_*`` functions mirror the C ABI of ``include/dasgd.h`` one to one
(raising ``DasgdError`` on a non-OK status); ``DaSGD`` is a small convenience wrapper that
allocates the caller-owned buffers as torch tensors.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

from . import build as _build

# ---------------------------------------------------------------- constants (include/dasgd.h)
DASGD_OK, DASGD_ERR_INVALID_ARG, DASGD_ERR_BAD_STATE, DASGD_ERR_NO_SLOT = 0, 1, 2, 3
DASGD_ERR_CUDA, DASGD_ERR_TIMEOUT, DASGD_ERR_UNSUPPORTED = 4, 5, 6
DASGD_F32, DASGD_BF16_MASTER_F32 = 0, 1
DASGD_MERGE_XI, DASGD_MERGE_DELTA = 0, 1
DASGD_FLAG_TIMING, DASGD_FLAG_FUSE_SNAPSHOT, DASGD_FLAG_FUSE_MERGE, DASGD_FLAG_ROTATE_SNAPSHOT = 0x1, 0x2, 0x4, 0x8
DASGD_FLAG_INLINE_MEAN = 0x10
DASGD_FLAG_NESTEROV, DASGD_FLAG_DECOUPLED_WD = 0x20, 0x40
DASGD_FLAG_FUSE_MERGE_D1 = 0x80
DASGD_FLAG_TWO_LANES = 0x100
DASGD_FLAG_GRAPH = 0x200
DASGD_FLAG_TWO_SIDE_STREAMS = 0x400

EXPORTS = [
    "dasgd_init", "dasgd_local_step", "dasgd_snapshot", "dasgd_average_async", "dasgd_merge", "dasgd_sync",
    "dasgd_step", "dasgd_step_host", "dasgd_get_weights", "dasgd_get_step", "dasgd_get_pending", "dasgd_get_timing",
    "dasgd_get_kernel_timing", "dasgd_reset_timing", "dasgd_get_launches", "dasgd_strerror", "dasgd_last_error", "dasgd_destroy", "dasgd_version",
    "dasgd_average_merge_noalloc", "dasgd_delay_guideline", "dasgd_advise_delay", "dasgd_export_state", "dasgd_import_state",
    "dasgd_get_kernel_units", "dasgd_refresh_lp",
    "dasgd_set_momentum_averaging", "dasgd_get_pending_momentum",
    "dasgd_set_shard", "dasgd_set_shard_nccl", "dasgd_nccl_unique_id", "dasgd_nccl_comm_init", "dasgd_nccl_comm_destroy",
]

# dasgd_exchange_fn: (user, send_device, recv_device, count, side_stream) -> status
EXCHANGE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p)


class dasgd_config(ctypes.Structure):
    _fields_ = [
        ("K", ctypes.c_int32), ("tau", ctypes.c_int32), ("d", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("merge_mode", ctypes.c_int32), ("n_slots", ctypes.c_int32), ("flags", ctypes.c_uint32),
        ("device", ctypes.c_int32), ("P", ctypes.c_int64), ("ld", ctypes.c_int64),
        ("xi", ctypes.c_float), ("momentum", ctypes.c_float), ("weight_decay", ctypes.c_float),
        ("sync_timeout_ms", ctypes.c_uint32), ("n_stage", ctypes.c_int32), ("n_chunks", ctypes.c_int32),
        ("w", ctypes.c_void_p), ("m", ctypes.c_void_p), ("w_lp", ctypes.c_void_p), ("snap", ctypes.c_void_p),
        ("mean", ctypes.c_void_p), ("g_stage", ctypes.c_void_p),
        ("main_stream", ctypes.c_void_p), ("side_stream", ctypes.c_void_p),
    ]


class DasgdError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"libdasgd status {status}: {text}")
        self.status = status


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()  # raises if nvcc is unavailable
    L = ctypes.CDLL(path)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    L.dasgd_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(dasgd_config)]
    L.dasgd_local_step.argtypes = [vp, vp, f32]
    L.dasgd_snapshot.argtypes = [vp]
    L.dasgd_average_async.argtypes = [vp]
    L.dasgd_merge.argtypes = [vp]
    L.dasgd_sync.argtypes = [vp]
    L.dasgd_step.argtypes = [vp, vp, f32]
    L.dasgd_step_host.argtypes = [vp, vp, f32, vp, i64]
    L.dasgd_get_step.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i32)]
    L.dasgd_get_weights.argtypes = [vp, ctypes.POINTER(vp)]
    L.dasgd_get_pending.argtypes = [vp, i32, ctypes.POINTER(i64), ctypes.POINTER(vp), ctypes.POINTER(vp)]
    L.dasgd_get_timing.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(ctypes.c_double),
                                   ctypes.POINTER(ctypes.c_double)]
    L.dasgd_get_launches.argtypes = [vp, ctypes.POINTER(i64)]
    L.dasgd_get_kernel_timing.argtypes = [vp, i32, ctypes.POINTER(i64), ctypes.POINTER(ctypes.c_double)]
    L.dasgd_get_kernel_units.argtypes = [vp, i32, ctypes.POINTER(i64)]
    L.dasgd_refresh_lp.argtypes = [vp]
    L.dasgd_reset_timing.argtypes = [vp]
    L.dasgd_strerror.argtypes = [ctypes.c_int]
    L.dasgd_strerror.restype = ctypes.c_char_p
    L.dasgd_last_error.argtypes = [vp]
    L.dasgd_last_error.restype = ctypes.c_char_p
    L.dasgd_destroy.argtypes = [vp]
    L.dasgd_average_merge_noalloc.argtypes = [vp, i32, i64, i64, f32, i32, vp, ctypes.c_char_p, i64]
    f64, pi32, pf64 = ctypes.c_double, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double)
    L.dasgd_delay_guideline.argtypes = [f64, f64, pi32, pi32]
    L.dasgd_advise_delay.argtypes = [vp, f64, pi32, pi32, pf64, pf64]
    L.dasgd_export_state.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
    L.dasgd_import_state.argtypes = [vp, vp, i64]
    L.dasgd_set_momentum_averaging.argtypes = [vp, vp, vp]
    L.dasgd_get_pending_momentum.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    L.dasgd_set_shard.argtypes = [vp, i32, EXCHANGE_FN, vp]
    L.dasgd_set_shard_nccl.argtypes = [vp, i32, vp]
    L.dasgd_nccl_unique_id.argtypes = [vp]
    L.dasgd_nccl_comm_init.argtypes = [ctypes.POINTER(vp), vp, i32, i32, i32]
    L.dasgd_nccl_comm_destroy.argtypes = [vp]
    L.dasgd_version.argtypes = []
    L.dasgd_version.restype = ctypes.c_char_p
    return L


_L = _load()


def _check(status: int, ctx=None):
    if status != DASGD_OK:
        detail = _L.dasgd_last_error(ctx).decode() if (ctx or status) else ""
        raise DasgdError(status, f"{_L.dasgd_strerror(status).decode()}: {detail}")


# ---------------------------------------------------------------- the C ABI, name for name

def dasgd_version() -> str:
    return _L.dasgd_version().decode()


def dasgd_init(cfg: dasgd_config) -> ctypes.c_void_p:
    ctx = ctypes.c_void_p()
    _check(_L.dasgd_init(ctypes.byref(ctx), ctypes.byref(cfg)), None)
    return ctx


def dasgd_local_step(ctx, grads_ptr: int, lr: float):
    _check(_L.dasgd_local_step(ctx, grads_ptr, lr), ctx)


def dasgd_snapshot(ctx):
    _check(_L.dasgd_snapshot(ctx), ctx)


def dasgd_average_async(ctx):
    _check(_L.dasgd_average_async(ctx), ctx)


def dasgd_merge(ctx):
    _check(_L.dasgd_merge(ctx), ctx)


def dasgd_sync(ctx):
    _check(_L.dasgd_sync(ctx), ctx)


def dasgd_step(ctx, grads_ptr: int, lr: float):
    _check(_L.dasgd_step(ctx, grads_ptr, lr), ctx)


def dasgd_step_host(ctx, grads_host_ptr: int, lr: float, probe_host_ptr: int | None, probe_elems: int):
    _check(_L.dasgd_step_host(ctx, grads_host_ptr, lr, probe_host_ptr, probe_elems), ctx)


def dasgd_get_weights(ctx) -> int:
    w = ctypes.c_void_p()
    _check(_L.dasgd_get_weights(ctx, ctypes.byref(w)), ctx)
    return w.value


def dasgd_get_step(ctx):
    t, pend = ctypes.c_int64(), ctypes.c_int32()
    _check(_L.dasgd_get_step(ctx, ctypes.byref(t), ctypes.byref(pend)), ctx)
    return t.value, pend.value


def dasgd_get_pending(ctx, i: int):
    s, snap, mean = ctypes.c_int64(), ctypes.c_void_p(), ctypes.c_void_p()
    _check(_L.dasgd_get_pending(ctx, i, ctypes.byref(s), ctypes.byref(snap), ctypes.byref(mean)), ctx)
    return s.value, snap.value, mean.value


def dasgd_get_timing(ctx):
    n, a, st = ctypes.c_int64(), ctypes.c_double(), ctypes.c_double()
    _check(_L.dasgd_get_timing(ctx, ctypes.byref(n), ctypes.byref(a), ctypes.byref(st)), ctx)
    return n.value, a.value, st.value


def dasgd_get_kernel_timing(ctx, which: int):
    n, ms = ctypes.c_int64(), ctypes.c_double()
    _check(_L.dasgd_get_kernel_timing(ctx, which, ctypes.byref(n), ctypes.byref(ms)), ctx)
    return n.value, ms.value


def dasgd_get_kernel_units(ctx, which: int) -> int:
    n = ctypes.c_int64()
    _check(_L.dasgd_get_kernel_units(ctx, which, ctypes.byref(n)), ctx)
    return n.value


def dasgd_refresh_lp(ctx):
    _check(_L.dasgd_refresh_lp(ctx), ctx)


def dasgd_reset_timing(ctx):
    _check(_L.dasgd_reset_timing(ctx), ctx)


def dasgd_delay_guideline(t_c: float, t_p: float):
    """(d, tau): smallest d with t_c < d*t_p, tau = d + 1 (the paper's guideline, Eq. 3)."""
    d, tau = ctypes.c_int32(), ctypes.c_int32()
    st = _L.dasgd_delay_guideline(t_c, t_p, ctypes.byref(d), ctypes.byref(tau))
    if st != DASGD_OK:
        raise DasgdError(st, "delay_guideline: need t_c >= 0 and t_p > 0")
    return d.value, tau.value


def dasgd_advise_delay(ctx, extra_tp_ms: float = 0.0):
    """(d, tau, t_c_ms, t_p_ms) from the context's own timings (needs DASGD_FLAG_TIMING)."""
    d, tau, tc, tp = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_double(), ctypes.c_double()
    _check(_L.dasgd_advise_delay(ctx, extra_tp_ms, ctypes.byref(d), ctypes.byref(tau), ctypes.byref(tc),
                                 ctypes.byref(tp)), ctx)
    return d.value, tau.value, tc.value, tp.value


def dasgd_export_state(ctx) -> bytes:
    buf, n = ctypes.create_string_buffer(4096), ctypes.c_int64()
    _check(_L.dasgd_export_state(ctx, buf, len(buf), ctypes.byref(n)), ctx)
    return buf.raw[:n.value]


def dasgd_import_state(ctx, blob: bytes):
    _check(_L.dasgd_import_state(ctx, blob, len(blob)), ctx)


def dasgd_set_momentum_averaging(ctx, m_snap_ptr: int, m_mean_ptr: int):
    _check(_L.dasgd_set_momentum_averaging(ctx, m_snap_ptr, m_mean_ptr), ctx)


def dasgd_get_pending_momentum(ctx, i: int):
    snap, mean = ctypes.c_void_p(), ctypes.c_void_p()
    _check(_L.dasgd_get_pending_momentum(ctx, i, ctypes.byref(snap), ctypes.byref(mean)), ctx)
    return snap.value, mean.value


def dasgd_set_shard(ctx, K_total: int, exchange, user=None):
    """`exchange`: an EXCHANGE_FN instance; the caller keeps it alive as long as the context."""
    _check(_L.dasgd_set_shard(ctx, K_total, exchange, user), ctx)


def dasgd_set_shard_nccl(ctx, K_total: int, comm):
    _check(_L.dasgd_set_shard_nccl(ctx, K_total, comm), ctx)


def dasgd_nccl_unique_id() -> bytes:
    buf = ctypes.create_string_buffer(128)
    _check(_L.dasgd_nccl_unique_id(buf), None)
    return buf.raw


def dasgd_nccl_comm_init(unique_id: bytes, nranks: int, rank: int, device: int) -> ctypes.c_void_p:
    comm = ctypes.c_void_p()
    _check(_L.dasgd_nccl_comm_init(ctypes.byref(comm), unique_id, nranks, rank, device), None)
    return comm


def dasgd_nccl_comm_destroy(comm):
    _check(_L.dasgd_nccl_comm_destroy(comm), None)


def dasgd_get_launches(ctx) -> int:
    n = ctypes.c_int64()
    _check(_L.dasgd_get_launches(ctx, ctypes.byref(n)), ctx)
    return n.value


def dasgd_destroy(ctx):
    _check(_L.dasgd_destroy(ctx), None)


DASGD_NOALLOC_MAX_P = 1 << 20


def dasgd_average_merge_noalloc(w_ptr: int, K: int, P: int, ld: int, xi: float, device: int, stream_ptr: int | None):
    """Average the K rows of w and blend the mean back (xi*w + (1-xi)*mean) using only the library's
    built-in 4 MiB mean vector: for callers that must not allocate device memory.  P is limited to
    DASGD_NOALLOC_MAX_P; calls that may overlap on the GPU must be ordered by the caller."""
    buf = ctypes.create_string_buffer(256)
    st = _L.dasgd_average_merge_noalloc(w_ptr, K, P, ld, xi, device, stream_ptr, buf, len(buf))
    if st != DASGD_OK:
        raise DasgdError(st, f"{_L.dasgd_strerror(st).decode()}: {buf.value.decode()}")


# ---------------------------------------------------------------- convenience wrapper

def min_slots(tau: int, d: int) -> int:
    return max(1, math.ceil(d / tau))


class DaSGD:
    """K replicas of a P-vector on one GPU.  Owns the torch tensors and streams the library borrows.

    ``w``, ``m`` are ``[K, ld]`` float32 tensors (``[:, :P]`` is the payload); in bf16 mode ``w_lp``
    is the ``[K, ld]`` bfloat16 copy.  ``main`` / ``side`` are the two torch streams.
    """

    def __init__(self, K, P, tau, d, xi, momentum=0.0, weight_decay=0.0, dtype=DASGD_F32,
                 merge_mode=DASGD_MERGE_XI, flags=0, n_slots=None, ld=None, device=0, host_staging=False,
                 sync_timeout_ms=0, order_after_current=True, snapshot_arrays=True, n_chunks=0, average_momentum=False):
        if not torch.cuda.is_available():
            raise RuntimeError("DaSGD needs a CUDA device; there is no CPU implementation")
        self.K, self.P, self.tau, self.d = K, P, tau, d
        self.dtype = dtype
        # True: before each step the main stream is made to wait (on the device) for torch's current
        # stream, so gradients just produced by torch ops are complete.  Costs one event per call.
        self.order_after_current = order_after_current
        self.device = torch.device("cuda", device)
        self.ld = ld if ld is not None else P
        self.n_slots = n_slots if n_slots is not None else min_slots(tau, d)
        dev = self.device
        self.gdtype = torch.bfloat16 if dtype == DASGD_BF16_MASTER_F32 else torch.float32
        self._w0 = torch.zeros((K, self.ld), dtype=torch.float32, device=dev)
        self.m = torch.zeros((K, self.ld), dtype=torch.float32, device=dev) if momentum != 0.0 else None
        self.w_lp = torch.zeros((K, self.ld), dtype=torch.bfloat16, device=dev) if dtype == DASGD_BF16_MASTER_F32 else None
        # the inline-mean schedule never touches snapshot arrays; they can be left out to save memory
        self.snap = (torch.empty((self.n_slots, K, self.ld), dtype=torch.float32, device=dev)
                     if snapshot_arrays or not (flags & DASGD_FLAG_INLINE_MEAN) else None)
        self.mean = torch.empty((self.n_slots, self.ld), dtype=torch.float32, device=dev)
        n_stage = int(host_staging) if host_staging in (0, 1, 2, True, False) else 0
        self.g_stage = torch.empty((n_stage, K, self.ld), dtype=self.gdtype, device=dev) if n_stage else None
        try:
            lo, hi = torch.cuda.Stream.priority_range()  # (least, greatest) priority
        except Exception:
            lo, hi = 0, -1
        self.main = torch.cuda.Stream(device=dev, priority=lo)
        self.side = torch.cuda.Stream(device=dev, priority=hi)
        cfg = dasgd_config()
        cfg.K, cfg.tau, cfg.d, cfg.dtype, cfg.merge_mode = K, tau, d, dtype, merge_mode
        cfg.n_slots, cfg.flags, cfg.device, cfg.P, cfg.ld = self.n_slots, flags, dev.index or 0, P, self.ld
        cfg.xi, cfg.momentum, cfg.weight_decay, cfg.sync_timeout_ms = xi, momentum, weight_decay, sync_timeout_ms
        cfg.w = self._w0.data_ptr()
        cfg.m = self.m.data_ptr() if self.m is not None else None
        cfg.w_lp = self.w_lp.data_ptr() if self.w_lp is not None else None
        cfg.snap = self.snap.data_ptr() if self.snap is not None else None
        cfg.mean = self.mean.data_ptr()
        cfg.g_stage = self.g_stage.data_ptr() if self.g_stage is not None else None
        cfg.n_stage = n_stage
        cfg.n_chunks = n_chunks
        cfg.main_stream, cfg.side_stream = self.main.cuda_stream, self.side.cuda_stream
        self.cfg = cfg
        self._host_refs = []
        torch.cuda.synchronize(dev)  # the zero fills above ran on torch's current stream
        self.ctx = dasgd_init(cfg)
        self.m_snap = self.m_mean = None
        if average_momentum:   # the variant in which the momentum buffers are averaged like the weights
            self.m_snap = torch.empty((self.n_slots, K, self.ld), dtype=torch.float32, device=dev)
            self.m_mean = torch.empty((self.n_slots, self.ld), dtype=torch.float32, device=dev)
            try:
                dasgd_set_momentum_averaging(self.ctx, self.m_snap.data_ptr(), self.m_mean.data_ptr())
            except DasgdError:
                self.close()
                raise

    # -- state ---------------------------------------------------------------
    @property
    def w(self) -> torch.Tensor:
        """The [K, ld] float32 array that holds the current weights (it moves between arrays when
        DASGD_FLAG_ROTATE_SNAPSHOT is set; fetch it again after every call that writes weights)."""
        ptr = dasgd_get_weights(self.ctx)
        if ptr == self._w0.data_ptr():
            return self._w0
        slot = (ptr - self.snap.data_ptr()) // (self.K * self.ld * 4)
        return self.snap[slot]

    def set_state(self, w, m=None):
        """Copy initial weights ([P] shared start or [K, P]) and optionally momentum into the buffers."""
        self.sync()  # work already queued on the library's streams must not race with the copies below
        w = torch.as_tensor(w, dtype=torch.float32, device=self.device)
        self.w[:, :self.P] = w if w.dim() == 2 else w.unsqueeze(0)
        if m is not None and self.m is not None:
            self.m[:, :self.P] = torch.as_tensor(m, dtype=torch.float32, device=self.device)
        torch.cuda.synchronize(self.device)
        if self.w_lp is not None:
            dasgd_refresh_lp(self.ctx)  # the library's own float32 -> bfloat16 rounding, on the main stream
            self.sync()

    def _gptr(self, g: torch.Tensor) -> int:
        if self.order_after_current:
            self.main.wait_stream(torch.cuda.current_stream(self.device))
        if g.dtype != self.gdtype or tuple(g.shape) != (self.K, self.ld) or not g.is_contiguous() or not g.is_cuda:
            raise ValueError(f"gradients must be a contiguous CUDA {self.gdtype} tensor of shape {(self.K, self.ld)}")
        # The kernels read g on the library's main stream, not on the stream torch allocated it on.  Telling
        # the caching allocator keeps the block from being handed out again while they may still read it, so
        # callers may pass temporaries (``eng.step(g_host.cuda(), lr)``).
        g.record_stream(self.main)
        return g.data_ptr()

    # -- the path --------------------------------------------------------------
    def local_step(self, g, lr):
        dasgd_local_step(self.ctx, self._gptr(g), lr)

    def snapshot(self):
        dasgd_snapshot(self.ctx)

    def average_async(self):
        dasgd_average_async(self.ctx)

    def merge(self):
        dasgd_merge(self.ctx)

    def sync(self):
        dasgd_sync(self.ctx)
        self._host_refs.clear()

    def step(self, g, lr):
        dasgd_step(self.ctx, self._gptr(g), lr)

    def step_host(self, g_host: torch.Tensor, lr, probe_host: torch.Tensor | None = None):
        if g_host.is_cuda or g_host.dtype != self.gdtype or tuple(g_host.shape) != (self.K, self.ld):
            raise ValueError("step_host wants a host tensor shaped like the gradients")
        n = probe_host.numel() if probe_host is not None else 0
        # the asynchronous copies read / write these host tensors until the next sync: keep them alive
        self._host_refs.append((g_host, probe_host))
        dasgd_step_host(self.ctx, g_host.data_ptr(), lr, probe_host.data_ptr() if n else None, n)

    # -- introspection ---------------------------------------------------------
    @property
    def t(self):
        return dasgd_get_step(self.ctx)[0]

    @property
    def n_pending(self):
        return dasgd_get_step(self.ctx)[1]

    def pending_mean(self, i=0) -> torch.Tensor:
        """The mean vector of the i-th oldest pending snapshot (a view into ``self.mean``)."""
        _, _, mean_ptr = dasgd_get_pending(self.ctx, i)
        slot = (mean_ptr - self.mean.data_ptr()) // (self.ld * 4)
        return self.mean[slot, :self.P]

    def pending_momentum_mean(self, i=0) -> torch.Tensor:
        """The mean of the momentum buffers of the i-th oldest pending snapshot (momentum averaging only)."""
        _, mean_ptr = dasgd_get_pending_momentum(self.ctx, i)
        slot = (mean_ptr - self.m_mean.data_ptr()) // (self.ld * 4)
        return self.m_mean[slot, :self.P]

    def timing(self):
        """(averages completed, ms spent averaging on the side stream, ms the main stream waited for them)."""
        return dasgd_get_timing(self.ctx)

    KERNELS = ("local_step", "snapshot", "mean", "merge", "stall")

    def kernel_timing(self):
        """{kind: (launches, total ms)} for the five kinds of timed work."""
        return {name: dasgd_get_kernel_timing(self.ctx, i) for i, name in enumerate(self.KERNELS)}

    def kernel_units(self):
        """{kind: replica-parameters processed by the timed launches of that kind}."""
        return {name: dasgd_get_kernel_units(self.ctx, i) for i, name in enumerate(self.KERNELS)}

    def reset_timing(self):
        dasgd_reset_timing(self.ctx)

    def state_dict(self) -> dict:
        """Everything needed to resume: the schedule blob and copies of the device arrays."""
        blob = dasgd_export_state(self.ctx)       # synchronises both streams
        out = {"schedule": blob, "w0": self._w0.clone(), "mean": self.mean.clone()}
        for name in ("m", "w_lp", "snap"):
            t = getattr(self, name)
            out[name] = t.clone() if t is not None else None
        torch.cuda.synchronize(self.device)
        return out

    def load_state_dict(self, sd: dict):
        """Into a freshly built object of the same configuration."""
        self.sync()
        self._w0.copy_(sd["w0"]); self.mean.copy_(sd["mean"])
        for name in ("m", "w_lp", "snap"):
            if getattr(self, name) is not None and sd[name] is not None:
                getattr(self, name).copy_(sd[name])
        torch.cuda.synchronize(self.device)
        dasgd_import_state(self.ctx, sd["schedule"])

    def advise_delay(self, extra_tp_ms=0.0):
        return dasgd_advise_delay(self.ctx, extra_tp_ms)

    @property
    def launches(self):
        return dasgd_get_launches(self.ctx)

    # -- sharded worker axis ---------------------------------------------------
    def set_shard(self, K_total, exchange=None, nccl_comm=None):
        """This object holds K of K_total workers.  Either `nccl_comm` (from dasgd_nccl_comm_init) or
        `exchange(send_ptr, recv_ptr, count, stream_ptr)`, a Python callable that enqueues the all-reduce of
        the partial sums on the side stream."""
        if nccl_comm is not None:
            dasgd_set_shard_nccl(self.ctx, K_total, nccl_comm)
        else:
            def thunk(user, send, recv, count, stream):
                try:
                    exchange(send, recv, count, stream)
                    return DASGD_OK
                except Exception:
                    return DASGD_ERR_CUDA
            self._exchange = EXCHANGE_FN(thunk)      # keep the callback object alive
            dasgd_set_shard(self.ctx, K_total, self._exchange, None)
        self.K_total = K_total

    def close(self):
        if getattr(self, "ctx", None):
            dasgd_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
