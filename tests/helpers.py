"""Shared test plumbing: drives the CUDA library and the CPU oracle over the same seeded event
stream and compares them.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

REL_ONE_STEP = 1e-5      # max relative error after one update
REL_100_STEPS = 1e-4     # max relative error after 100 updates


def rel_err(got, want):
    """max_k |got - want| / max(|want_k|, rms(want)): relative error that stays defined near zero."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    rms = float(np.sqrt(np.mean(want * want))) if want.size else 0.0
    den = np.maximum(np.abs(want), max(rms, 1e-30))
    return float(np.max(np.abs(got - want) / den)) if want.size else 0.0


def adagrad_slack(h_oracle, abar, terms, gmax, eps=1e-8):
    """Absolute error one AdaGrad step may add to a weight beyond the relative bar, per weight.

    The step is abar * g / (sqrt(h) + eps) with h the running sum of squares including g^2; its
    derivative with respect to g is at most abar / (sqrt(h) + eps).  An fp32 evaluation of g (a mean
    of `terms` values of magnitude up to gmax plus the penalty) is off by up to about
    (terms + 2) 2^-24 gmax, which the division amplifies where sqrt(h) is small -- in the first
    steps, for the few weights whose gradient happens to be within a few hundred eps of zero.
    h_oracle is the oracle's state after the step."""
    delta = (terms + 2) * 2.0 ** -24 * gmax
    return abar * delta / (np.sqrt(np.asarray(h_oracle, dtype=np.float64)) + eps)


def rel_err_beyond(got, want, slack):
    """rel_err after an absolute allowance ``slack`` (per weight) has been taken off the difference."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    rms = float(np.sqrt(np.mean(want * want)))
    den = np.maximum(np.abs(want), max(rms, 1e-30))
    return float(np.max(np.maximum(np.abs(got - want) - slack, 0.0) / den))


def to_device(arr):
    """numpy -> CUDA tensor holding the same bytes (uint16 bf16 patterns travel as int16)."""
    import torch

    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    return torch.from_numpy(a).cuda()


def to_host(t):
    return t.detach().cpu().numpy()


class Pair:
    """A CUDA parameter server and an oracle server fed the same bytes."""

    def __init__(self, N, lam, n, alpha0, momentum=0.0, wd=0.0, dtype=synth.GRAD_F32, policy=0, optimizer=0,
                 theta0=None, seed=synth.MASTER_SEED):
        import torch
        from paper_1509_04210_b200 import binding as rb

        self.rb, self.torch = rb, torch
        self.N, self.lam, self.n, self.c = N, lam, n, lam // n
        self.dtype, self.momentum, self.optimizer = dtype, momentum, optimizer
        self.gpu = rb.ParameterServer(N, lam, n, alpha0, momentum, wd)
        self.cpu = ora.OraclePS(N, lam, n, alpha0, momentum, wd)
        if dtype != synth.GRAD_F32:
            self.gpu.set_option(rb.OPT_GRAD_DTYPE, dtype)
            self.cpu.set_grad_dtype(dtype)
        if policy:
            self.gpu.set_option(rb.OPT_LR_POLICY, policy)
            self.cpu.set_policy(policy)
        if optimizer:
            self.gpu.set_option(rb.OPT_OPTIMIZER, optimizer)
            self.cpu.set_optimizer(optimizer, 1e-8)
        th0 = synth.initial_weights(N, 0.01, seed) if theta0 is None else theta0
        self.theta0 = th0
        self.gpu.set_weights(to_device(th0))
        self.cpu.set_weights(th0)
        self._alive = []

    def push(self, grad_np, pulled_ts):
        g = to_device(grad_np)
        self._alive.append(g)
        a = self.gpu.push(g, pulled_ts)
        b = self.cpu.push(grad_np, pulled_ts)
        assert a == b, (a, b)
        return a

    def step(self, dsts=None):
        a = self.gpu.step() if dsts is None else self.gpu.step_pull_many(dsts)
        b = self.cpu.step()
        assert a == b, (a, b)
        if a == 1:
            self.gpu.sync()
            del self._alive[: self.c]
            self.check_clock()
        return a

    def check_clock(self):
        g, o = self.gpu.last_clock(), self.cpu.last_clock()
        assert g["c"] == o["c"] == self.c
        np.testing.assert_array_equal(g["pulled_ts"], o["pulled_ts"])
        np.testing.assert_array_equal(g["sigma"], o["sigma"])
        np.testing.assert_array_equal(g["scale"].view(np.uint32), o["scale"].view(np.uint32))
        assert g["avg_sigma"] == o["avg_sigma"]
        assert self.gpu.timestamp() == self.cpu.timestamp()

    def weights(self):
        t = self.torch.empty(self.N, dtype=self.torch.float32, device="cuda")
        s = self.torch.empty(self.N, dtype=self.torch.float32, device="cuda")
        self.gpu.export_state(t, s)
        self.gpu.sync()
        return to_host(t), to_host(s)

    def compare(self, tol):
        th_g, st_g = self.weights()
        th_o, ts = self.cpu.pull()
        st_o = self.cpu.state()
        e_th = rel_err(th_g, th_o)
        assert e_th <= tol, ("weights", e_th, tol)
        if self.momentum != 0.0 or self.optimizer != 0:
            e_st = rel_err(st_g, st_o)
            assert e_st <= tol, ("state", e_st, tol)
        return e_th

    def close(self):
        self.gpu.close()


def run_workload(w: synth.Workload, updates, check_every=1, N=None, seed=synth.MASTER_SEED, policy=0, fused_pull=False):
    """Replays ``updates`` weight updates of workload w through both servers, event by event,
    checking integers bit-exactly at every update and weights every ``check_every`` updates.
    Returns the list of (update index, relative error)."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = w.nparams if N is None else N
    pair = Pair(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay, w.grad_dtype, policy, seed=seed)
    gs = rb.Scheduler(w.lam, w.n, w.mode, seed, w.lognormal_sigma, w.downcast)
    os_ = ora.OracleScheduler(w.lam, w.n, w.mode, seed, w.lognormal_sigma, w.downcast)
    slots = [torch.zeros(N, dtype=torch.float32, device="cuda") for _ in range(w.lam)]
    slot_ts = [0] * w.lam
    errs, done = [], 0
    pending_step = False
    while done < updates:
        ev = gs.next(1)[0]
        eo = os_.run(1)[0]
        assert ev.tobytes() == eo.tobytes(), (ev, eo)            # scheduling: bit-exact
        kind, l = int(ev["kind"]), int(ev["learner"])
        if kind == rb.EV_PUSH:
            assert int(ev["ts"]) == pair.gpu.timestamp()
            assert int(ev["pulled_ts"]) == slot_ts[l] or w.downcast
            g = synth.gradient(N, l, int(ev["seq"]), w.grad_std, w.grad_dtype, seed)
            pair.push(g, int(ev["pulled_ts"]))
        elif kind == rb.EV_STEP:
            if fused_pull and (w.downcast or w.mode == synth.HARDSYNC):
                pending_step = True       # the broadcast that follows is fused into the update
                continue
            assert pair.step() == 1
            assert pair.gpu.timestamp() == int(ev["ts"])
            done += 1
            tol = REL_ONE_STEP if done == 1 else REL_100_STEPS
            if done == 1 or done % check_every == 0 or done == updates:
                errs.append((done, pair.compare(tol)))
        elif kind == rb.EV_PULL:
            ts = pair.gpu.pull(slots[l])
            want, ts_o = pair.cpu.pull()
            assert ts == ts_o == int(ev["ts"])
            slot_ts[l] = ts
            pair.gpu.sync()
            if done % check_every == 0:
                th, _ = pair.weights()
                np.testing.assert_array_equal(to_host(slots[l]), th)   # a pull is an exact copy
        elif kind == rb.EV_PULL_SKIP:
            assert pair.gpu.timestamp() == int(ev["ts"])
        elif kind == rb.EV_BROADCAST:
            if pending_step:
                assert pair.step(dsts=slots) == 1
                pending_step = False
                done += 1
                tol = REL_ONE_STEP if done == 1 else REL_100_STEPS
                errs.append((done, pair.compare(tol)))
            else:
                ts = pair.gpu.pull_many(slots)
                assert ts == int(ev["ts"])
            pair.gpu.sync()
            slot_ts = [int(ev["ts"])] * w.lam
            if done % check_every == 0:
                th, _ = pair.weights()
                for s in (slots[0], slots[-1], slots[len(slots) // 2]):
                    np.testing.assert_array_equal(to_host(s), th)
    pair.close()
    return errs
