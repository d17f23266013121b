"""ctypes access to the C++ oracle in ``rudra_oracle.cpp`` (test infrastructure, not product code).

The arithmetic lives in the C++ file; this module only compiles it with g++ and marshals
numpy arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rudra_oracle.cpp")
_LIB = os.path.join(_HERE, "librudra_oracle.so")

# event kinds / scheduler modes / options: integer values fixed by the event contract
PUSH, STEP, PULL, PULL_SKIP, BROADCAST, RELAY = 1, 2, 3, 4, 5, 6
HARDSYNC, SOFTSYNC_ROUNDS, SOFTSYNC_TIMED = 0, 1, 2
LR_PAPER_N, LR_PER_GRADIENT, LR_GROUP_MEAN = 0, 1, 2
GRAD_F32, GRAD_BF16 = 0, 1
OPT_MOMENTUM_SGD, OPT_ADAGRAD = 0, 1

EVENT_DTYPE = np.dtype(
    [("kind", "<i4"), ("learner", "<u4"), ("pulled_ts", "<u8"), ("ts", "<u8"), ("seq", "<u8"), ("tick", "<u8")]
)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.ora_splitmix64.argtypes = [C.c_uint64, C.c_uint64, C.c_void_p]
        L.ora_sched_create.restype = C.c_void_p
        L.ora_sched_create.argtypes = [C.c_uint32, C.c_uint32, C.c_int32, C.c_uint64, C.c_double, C.c_int32]
        L.ora_sched_create_tree.restype = C.c_void_p
        L.ora_sched_create_tree.argtypes = [C.c_uint32, C.c_uint32, C.c_int32, C.c_uint64, C.c_double, C.c_int32, C.c_uint32]
        L.ora_sched_destroy.argtypes = [C.c_void_p]
        L.ora_sched_on_pull.restype = C.c_int32
        L.ora_sched_on_pull.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64]
        L.ora_sched_run.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        L.ora_ps_create.restype = C.c_void_p
        L.ora_ps_create.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_float, C.c_float, C.c_float]
        L.ora_ps_destroy.argtypes = [C.c_void_p]
        L.ora_ps_set_policy.argtypes = [C.c_void_p, C.c_int32]
        L.ora_ps_set_grad_dtype.argtypes = [C.c_void_p, C.c_int32]
        L.ora_ps_set_optimizer.argtypes = [C.c_void_p, C.c_int32, C.c_float]
        L.ora_ps_set_alpha0.argtypes = [C.c_void_p, C.c_float]
        L.ora_ps_set_strict.argtypes = [C.c_void_p, C.c_int32]
        L.ora_ps_set_weights.argtypes = [C.c_void_p, C.c_void_p]
        L.ora_ps_push.restype = C.c_int64
        L.ora_ps_push.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        L.ora_ps_push_relay.restype = C.c_int64
        L.ora_ps_push_relay.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32]
        L.ora_ps_last_messages.restype = C.c_int32
        L.ora_ps_last_messages.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.ora_ps_step.restype = C.c_int32
        L.ora_ps_step.argtypes = [C.c_void_p]
        L.ora_ps_pull.restype = C.c_int64
        L.ora_ps_pull.argtypes = [C.c_void_p, C.c_void_p]
        L.ora_ps_timestamp.restype = C.c_int64
        L.ora_ps_timestamp.argtypes = [C.c_void_p]
        L.ora_ps_state.argtypes = [C.c_void_p, C.c_void_p]
        L.ora_ps_last_clock.restype = C.c_int32
        L.ora_ps_last_clock.argtypes = [C.c_void_p] + [C.c_void_p] * 5
        _lib = L
    return _lib


def splitmix64(seed, count):
    out = np.zeros(count, dtype=np.uint64)
    lib().ora_splitmix64(seed, count, out.ctypes.data)
    return out


class OracleScheduler:
    """Event stream of lambda simulated learners (hardsync / n-softsync rounds / timed)."""

    def __init__(self, lam, n, mode=SOFTSYNC_ROUNDS, seed=20150914, lognormal_sigma=0.3, downcast=False, fanin=0):
        """fanin > 0: learners send to the leaves of a two-level server tree, fanin learners per leaf."""
        self._h = lib().ora_sched_create_tree(lam, n, mode, seed, float(lognormal_sigma), int(bool(downcast)), int(fanin))
        if not self._h:
            raise ValueError("invalid scheduler arguments")

    def run(self, count):
        ev = np.zeros(count, dtype=EVENT_DTYPE)
        lib().ora_sched_run(self._h, count, ev.ctypes.data)
        return ev

    def on_pull(self, learner, ts):
        """The learner really computes on weights with timestamp ``ts`` (a late or lost pull)."""
        return lib().ora_sched_on_pull(self._h, learner, ts)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().ora_sched_destroy(self._h)
            self._h = None


class OraclePS:
    """Parameter-server state and update rule on host memory, double arithmetic, fp32 storage."""

    def __init__(self, nparams, lam, n, alpha0, momentum, weight_decay):
        self.N, self.lam, self.n, self.c = int(nparams), int(lam), int(n), int(lam) // int(n)
        self._h = lib().ora_ps_create(nparams, lam, n, alpha0, momentum, weight_decay)
        if not self._h:
            raise ValueError("invalid parameter-server arguments")
        self._keep = []
        self._dtype = GRAD_F32

    def set_policy(self, policy):
        lib().ora_ps_set_policy(self._h, policy)

    def set_grad_dtype(self, dtype):
        self._dtype = dtype
        lib().ora_ps_set_grad_dtype(self._h, dtype)

    def set_optimizer(self, opt, eps=1e-8):
        lib().ora_ps_set_optimizer(self._h, opt, eps)

    def set_alpha0(self, a0):
        lib().ora_ps_set_alpha0(self._h, a0)

    def set_strict(self, on=True):
        """fp32 evaluation with one fused multiply-add per term (debugging aid, not the parity bar)."""
        lib().ora_ps_set_strict(self._h, int(bool(on)))

    def set_weights(self, theta0):
        a = np.ascontiguousarray(theta0, dtype=np.float32)
        assert a.size == self.N
        lib().ora_ps_set_weights(self._h, a.ctypes.data)
        self._keep.clear()

    def push(self, grad, pulled_ts):
        want = np.float32 if self._dtype == GRAD_F32 else np.uint16
        g = np.ascontiguousarray(grad)
        assert g.dtype == want and g.size == self.N, (g.dtype, g.size)
        r = lib().ora_ps_push(self._h, g.ctypes.data, int(pulled_ts))
        if r > 0:
            self._keep.append((1, g))  # the oracle reads the buffer when the group closes
        return r

    def push_relay(self, grads, pulled_ts):
        """A leaf of the server tree averages ``grads`` (arrival order) and relays the average."""
        want = np.float32 if self._dtype == GRAD_F32 else np.uint16
        gs = [np.ascontiguousarray(g) for g in grads]
        assert all(g.dtype == want and g.size == self.N for g in gs) and len(gs) == len(pulled_ts)
        table = (C.c_void_p * len(gs))(*[g.ctypes.data for g in gs])
        ts = np.ascontiguousarray(pulled_ts, dtype=np.uint64)
        r = lib().ora_ps_push_relay(self._h, table, ts.ctypes.data, len(gs))
        if r > 0:
            self._keep.append((len(gs), None))  # averaged at once: the leaf does not keep the gradients
        return r

    def step(self):
        r = lib().ora_ps_step(self._h)
        if r == 1:
            have = 0
            while have < self.c:
                have += self._keep.pop(0)[0]
        return r

    def last_messages(self):
        step = np.zeros(self.c, dtype=np.float32)
        fanin = np.zeros(self.c, dtype=np.uint32)
        m = lib().ora_ps_last_messages(self._h, step.ctypes.data, fanin.ctypes.data)
        return {"step": step[:m], "fanin": fanin[:m]}

    def pull(self):
        dst = np.empty(self.N, dtype=np.float32)
        ts = lib().ora_ps_pull(self._h, dst.ctypes.data)
        return dst, ts

    def timestamp(self):
        return lib().ora_ps_timestamp(self._h)

    def state(self):
        v = np.empty(self.N, dtype=np.float32)
        lib().ora_ps_state(self._h, v.ctypes.data)
        return v

    def last_clock(self):
        pulled = np.zeros(self.c, dtype=np.uint64)
        sigma = np.zeros(self.c, dtype=np.uint32)
        scale = np.zeros(self.c, dtype=np.float32)
        avg = C.c_double(0.0)
        abar = C.c_float(0.0)
        got = lib().ora_ps_last_clock(
            self._h, pulled.ctypes.data, sigma.ctypes.data, scale.ctypes.data, C.addressof(avg), C.addressof(abar)
        )
        return {"c": got, "pulled_ts": pulled[:got], "sigma": sigma[:got], "scale": scale[:got],
                "avg_sigma": avg.value, "abar": abar.value}

    def __del__(self):
        if getattr(self, "_h", None):
            lib().ora_ps_destroy(self._h)
            self._h = None
