"""Thin ctypes binding of ``include/rudra_ps.h``: argument marshalling only.

Every step of the path runs in the native library; this module never computes on weights or
gradients.  The library is loaded on first use.  If it is missing it is built with nvcc; if
that fails the import error is raised -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

# constants of include/rudra_ps.h
E_INVAL, E_BAD_TS, E_QUEUE_FULL, E_CUDA, E_STATE, E_NOMEM = -1, -2, -3, -4, -5, -6
MAX_GROUP, MAX_DSTS, QUEUE_CAP, HIST_BINS = 128, 128, 4096, 4096
OPT_GRAD_DTYPE, OPT_LR_POLICY, OPT_OPTIMIZER, OPT_PUSH_MODE, OPT_TREE_FANIN = 1, 2, 3, 4, 5
PUSH_BORROW, PUSH_COPY = 0, 1
GRAD_F32, GRAD_BF16 = 0, 1
LR_PAPER_N, LR_PER_GRADIENT, LR_GROUP_MEAN = 0, 1, 2
OPTIM_MOMENTUM_SGD, OPTIM_ADAGRAD = 0, 1
EV_PUSH, EV_STEP, EV_PULL, EV_PULL_SKIP, EV_BROADCAST, EV_RELAY = 1, 2, 3, 4, 5, 6
SCHED_HARDSYNC, SCHED_SOFTSYNC_ROUNDS, SCHED_SOFTSYNC_TIMED = 0, 1, 2

EVENT_DTYPE = np.dtype(
    [("kind", "<i4"), ("learner", "<u4"), ("pulled_ts", "<u8"), ("ts", "<u8"), ("seq", "<u8"), ("tick", "<u8")]
)


class RudraError(RuntimeError):
    def __init__(self, code, text):
        super().__init__("rudra_ps error %d: %s" % (code, text))
        self.code = code


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


def lib():
    """The loaded native library (built first if the in-tree .so is absent or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path) or _build.needs_build():
        try:
            _build.build()
        except Exception as exc:  # no nvcc and no prebuilt library: fail loudly
            if not os.path.exists(path):
                raise ImportError("librudra_ps.so is missing and could not be built: %r" % (exc,)) from exc
    L = C.CDLL(path)
    vp, u64, u32, i64, f32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int64, C.c_float
    sig = {
        "rudra_ps_create": (vp, [u64, u32, u32, f32, f32, f32]),
        "rudra_ps_destroy": (None, [vp]),
        "rudra_ps_set_stream": (C.c_int, [vp, vp]),
        "rudra_ps_set_option": (C.c_int, [vp, C.c_int, i64]),
        "rudra_ps_set_alpha0": (C.c_int, [vp, f32]),
        "rudra_ps_set_weights": (C.c_int, [vp, vp]),
        "rudra_ps_set_weights_host": (C.c_int, [vp, vp]),
        "rudra_ps_push": (i64, [vp, vp, u64]),
        "rudra_ps_push_host": (i64, [vp, vp, u64]),
        "rudra_ps_push_group": (i64, [vp, vp, u32, vp, u32]),
        "rudra_ps_last_messages": (C.c_int, [vp, vp, vp]),
        "rudra_leaf_average": (C.c_int, [vp, u32, C.c_int, u64, vp, vp]),
        "rudra_ps_step": (C.c_int, [vp]),
        "rudra_ps_step_pull_many": (C.c_int, [vp, vp, u32]),
        "rudra_ps_pull": (i64, [vp, vp]),
        "rudra_ps_pull_host": (i64, [vp, vp]),
        "rudra_ps_pull_many": (i64, [vp, vp, u32]),
        "rudra_ps_timestamp": (i64, [vp]),
        "rudra_ps_last_clock": (C.c_int, [vp, vp, vp, vp, vp]),
        "rudra_ps_export_state": (C.c_int, [vp, vp, vp]),
        "rudra_ps_import_state": (C.c_int, [vp, vp, vp, u64]),
        "rudra_ps_sync": (C.c_int, [vp]),
        "rudra_ps_counters": (C.c_int, [vp, vp]),
        "rudra_last_error": (C.c_char_p, []),
        "rudra_ps_update_host_noalloc": (C.c_int, [vp, vp, u64, vp, vp, u32, f32, f32, vp]),
        "rudra_noalloc_last_error": (C.c_char_p, []),
        "rudra_sched_create": (vp, [u32, u32, C.c_int, u64, C.c_double, C.c_int]),
        "rudra_sched_create_tree": (vp, [u32, u32, C.c_int, u64, C.c_double, C.c_int, u32]),
        "rudra_sched_on_pull": (C.c_int, [vp, u32, u64]),
        "rudra_sched_destroy": (None, [vp]),
        "rudra_sched_next": (i64, [vp, vp, u64]),
        "rudra_ps_run_events": (i64, [vp, vp, u64, vp, vp, u32]),
        "rudra_ps_clock_log": (i64, [vp, u64, u64, vp, vp]),
        "rudra_ps_staleness_histogram": (i64, [vp, vp, u32]),
        "rudra_ps_enable_views": (C.c_int, [vp, u32]),
        "rudra_ps_pull_view": (i64, [vp, u32, vp]),
        "rudra_ps_view_of": (i64, [vp, u32, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def last_error() -> str:
    return lib().rudra_last_error().decode()


def _check(code):
    if code < 0:
        raise RudraError(code, last_error())
    return code


def _ptr(x):
    """Address of a torch tensor, numpy array or raw integer."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError("expected a tensor, an ndarray or an address, got %r" % type(x))


def _ptr_array(xs):
    arr = (C.c_void_p * len(xs))(*[_ptr(x) for x in xs])
    return arr


def pointer_table(xs):
    """Host array of device addresses, reusable across calls."""
    return _ptr_array(xs)


NOALLOC_MAX_FLOATS = 4 * 1024 * 1024


def update_host_noalloc(theta_dev, state_dev, nparams, grads_host, scales, momentum, weight_decay, stream=None):
    """rudra_ps_update_host_noalloc: one fused update from host gradients, staged in the library's
    fixed device array instead of allocated buffers (for callers that must not allocate)."""
    c = len(grads_host)
    table = _ptr_array(grads_host)
    sc = np.ascontiguousarray(scales, dtype=np.float32)
    handle = stream.cuda_stream if hasattr(stream, "cuda_stream") else stream
    code = lib().rudra_ps_update_host_noalloc(_ptr(theta_dev), _ptr(state_dev), int(nparams), table, sc.ctypes.data, c,
                                              momentum, weight_decay, handle)
    if code < 0:
        raise RudraError(code, lib().rudra_noalloc_last_error().decode())
    return code


def leaf_average(grads_dev, grad_dtype, nparams, avg_dev, stream=None):
    """rudra_leaf_average: what a leaf of the server tree does to the gradients of its learners."""
    handle = stream.cuda_stream if hasattr(stream, "cuda_stream") else stream
    return _check(lib().rudra_leaf_average(_ptr_array(grads_dev), len(grads_dev), int(grad_dtype), int(nparams),
                                           _ptr(avg_dev), handle))


class Scheduler:
    """rudra_sched_*: the arrival order of push / pull messages of lambda simulated learners."""

    def __init__(self, lam, n, mode=SCHED_SOFTSYNC_ROUNDS, seed=20150914, lognormal_sigma=0.3, downcast=False, fanin=0):
        self._h = lib().rudra_sched_create_tree(lam, n, mode, seed, float(lognormal_sigma), int(bool(downcast)), int(fanin))
        if not self._h:
            raise ValueError("invalid scheduler arguments")

    def on_pull(self, learner, ts):
        return _check(lib().rudra_sched_on_pull(self._h, int(learner), int(ts)))

    def next(self, count):
        ev = np.zeros(count, dtype=EVENT_DTYPE)
        _check(lib().rudra_sched_next(self._h, ev.ctypes.data, count))
        return ev

    def close(self):
        if getattr(self, "_h", None):
            lib().rudra_sched_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:   # interpreter shutdown: the module may already be gone
            pass


class ParameterServer:
    """rudra_ps_*: one parameter server on the current CUDA device."""

    def __init__(self, nparams, lam, n, alpha0, momentum=0.0, weight_decay=0.0, stream=None):
        self.nparams, self.lam, self.n, self.c = int(nparams), int(lam), int(n), int(lam) // max(int(n), 1)
        self._h = lib().rudra_ps_create(nparams, lam, n, alpha0, momentum, weight_decay)
        if not self._h:
            raise RudraError(E_INVAL, last_error())
        if stream is not None:
            self.set_stream(stream)

    # -- configuration -----------------------------------------------------------------------
    def set_stream(self, stream):
        handle = stream.cuda_stream if hasattr(stream, "cuda_stream") else stream
        _check(lib().rudra_ps_set_stream(self._h, handle))

    def set_option(self, key, value):
        _check(lib().rudra_ps_set_option(self._h, key, value))

    def set_alpha0(self, alpha0):
        _check(lib().rudra_ps_set_alpha0(self._h, alpha0))

    def set_weights(self, src_dev):
        _check(lib().rudra_ps_set_weights(self._h, _ptr(src_dev)))

    def set_weights_host(self, src_host):
        _check(lib().rudra_ps_set_weights_host(self._h, _ptr(src_host)))

    # -- the path ----------------------------------------------------------------------------
    def push(self, grad_dev, pulled_ts):
        return _check(lib().rudra_ps_push(self._h, _ptr(grad_dev), int(pulled_ts)))

    def push_host(self, grad_host, pulled_ts):
        return _check(lib().rudra_ps_push_host(self._h, _ptr(grad_host), int(pulled_ts)))

    def push_group(self, vecs_dev, pulled_ts):
        """One message standing for len(pulled_ts) gradients: their average (one vector) or the raw vectors."""
        ts = np.ascontiguousarray(pulled_ts, dtype=np.uint64)
        return _check(lib().rudra_ps_push_group(self._h, _ptr_array(vecs_dev), len(vecs_dev), ts.ctypes.data, len(ts)))

    def last_messages(self):
        fanin = np.zeros(MAX_GROUP, dtype=np.uint32)
        step = np.zeros(MAX_GROUP, dtype=np.float32)
        m = _check(lib().rudra_ps_last_messages(self._h, fanin.ctypes.data, step.ctypes.data))
        return {"fanin": fanin[:m], "step": step[:m]}

    def step(self):
        return _check(lib().rudra_ps_step(self._h))

    def step_pull_many(self, dsts_dev):
        arr = _ptr_array(dsts_dev)
        return _check(lib().rudra_ps_step_pull_many(self._h, arr, len(dsts_dev)))

    def pull(self, dst_dev):
        return _check(lib().rudra_ps_pull(self._h, _ptr(dst_dev)))

    def pull_host(self, dst_host):
        return _check(lib().rudra_ps_pull_host(self._h, _ptr(dst_host)))

    def pull_many(self, dsts_dev):
        arr = _ptr_array(dsts_dev)
        return _check(lib().rudra_ps_pull_many(self._h, arr, len(dsts_dev)))

    def run_events(self, events, grads_dev, slots_dev=None, max_window=0):
        """events: array of EVENT_DTYPE; grads_dev / slots_dev: per-learner buffers (lists of tensors,
        or pointer tables made with ``pointer_table``)."""
        ev = np.ascontiguousarray(events, dtype=EVENT_DTYPE)
        g = grads_dev if isinstance(grads_dev, C.Array) else _ptr_array(grads_dev)
        sl = None if slots_dev is None else (slots_dev if isinstance(slots_dev, C.Array) else _ptr_array(slots_dev))
        return _check(lib().rudra_ps_run_events(self._h, ev.ctypes.data, len(ev), g, sl, int(max_window)))

    def run_events_at(self, events_address, count, grads_table, slots_table, max_window=0):
        """The same call for a caller that has marshalled its arguments once: the address of a
        contiguous EVENT_DTYPE array that it keeps alive, and pointer tables from ``pointer_table``."""
        code = _lib.rudra_ps_run_events(self._h, events_address, count, grads_table, slots_table, max_window)
        if code < 0:
            raise RudraError(code, last_error())
        return code

    def timestamp(self):
        return _check(lib().rudra_ps_timestamp(self._h))

    def last_clock(self):
        pulled = np.zeros(MAX_GROUP, dtype=np.uint64)
        sigma = np.zeros(MAX_GROUP, dtype=np.uint32)
        scale = np.zeros(MAX_GROUP, dtype=np.float32)
        avg = C.c_double(0.0)
        c = _check(lib().rudra_ps_last_clock(self._h, pulled.ctypes.data, sigma.ctypes.data, scale.ctypes.data,
                                             C.addressof(avg)))
        return {"c": c, "pulled_ts": pulled[:c], "sigma": sigma[:c], "scale": scale[:c], "avg_sigma": avg.value}

    def clock_log(self, first_ts, count):
        """(gradient timestamps [k, c], <sigma> [k]) of the updates first_ts, first_ts + 1, ..."""
        pulled = np.zeros((count, self.c), dtype=np.uint64)
        avg = np.zeros(count, dtype=np.float64)
        k = _check(lib().rudra_ps_clock_log(self._h, int(first_ts), int(count), pulled.ctypes.data, avg.ctypes.data))
        return pulled[:k], avg[:k]

    def staleness_histogram(self):
        need = _check(lib().rudra_ps_staleness_histogram(self._h, None, 0))
        counts = np.zeros(max(need, 1), dtype=np.uint64)
        _check(lib().rudra_ps_staleness_histogram(self._h, counts.ctypes.data, len(counts)))
        return counts[:need]

    def export_state(self, theta_dst_dev=None, state_dst_dev=None):
        _check(lib().rudra_ps_export_state(self._h, _ptr(theta_dst_dev), _ptr(state_dst_dev)))

    def import_state(self, theta_src_dev, state_src_dev, ts):
        _check(lib().rudra_ps_import_state(self._h, _ptr(theta_src_dev), _ptr(state_src_dev), int(ts)))

    def sync(self):
        _check(lib().rudra_ps_sync(self._h))

    def counters(self):
        out = np.zeros(8, dtype=np.uint64)
        _check(lib().rudra_ps_counters(self._h, out.ctypes.data))
        names = ("pushes", "updates", "pulls", "launches", "h2d_bytes", "d2h_bytes", "weight_copies", "versions")
        return dict(zip(names, (int(x) for x in out)))

    def enable_views(self, nversions):
        _check(lib().rudra_ps_enable_views(self._h, int(nversions)))

    def pull_view(self, learner):
        """(device address of the learner's new read-only weight vector, its timestamp)."""
        ptr = C.c_void_p(0)
        ts = _check(lib().rudra_ps_pull_view(self._h, int(learner), C.byref(ptr)))
        return ptr.value, ts

    def view_of(self, learner):
        ptr = C.c_void_p(0)
        ts = _check(lib().rudra_ps_view_of(self._h, int(learner), C.byref(ptr)))
        return ptr.value, ts

    def close(self):
        if getattr(self, "_h", None):
            lib().rudra_ps_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:   # interpreter shutdown: the module may already be gone
            pass
