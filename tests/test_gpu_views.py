"""Zero-copy pulls (weight versions shared by pointer, Section 3.3's buffer exchange applied to
learners on the server's GPU), through the C interface: every learner's view must hold the
oracle's weights as of the timestamp the view carries -- within tolerance of the double
evaluation, bit for bit the fp32 evaluation -- and, bit for bit, what a copying pull delivers."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, rel_err, to_device, to_host

pytestmark = pytest.mark.gpu


class _DevVector:
    """A device address as something torch can wrap without copying."""

    def __init__(self, ptr, n):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<f4", "data": (int(ptr), False), "version": 2}


def _view_tensor(ptr, n):
    import torch

    return torch.as_tensor(_DevVector(ptr, n), device="cuda")


def _servers(w, N, nversions):
    import torch
    from paper_1509_04210_b200 import binding as rb

    th0_np = synth.initial_weights(N, w.theta_std, 9)
    th0 = to_device(th0_np)
    grads_np = [synth.gradient(N, l, 0, w.grad_std, w.grad_dtype, 9) for l in range(w.lam)]
    grads = [to_device(g) for g in grads_np]
    out = []
    for _ in range(2):
        ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
        ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
        ps.set_weights(th0)
        out.append(ps)
    out[1].enable_views(nversions)
    slots = [torch.full((N,), -1.0, device="cuda") for _ in range(w.lam)]
    return rb, out[0], out[1], grads, slots, (th0_np, grads_np)


@pytest.mark.parametrize("name,N,nevents", [("imagenet", 30011, 1500), ("imagenet", 280003, 600), ("cifar10", 9001, 900), ("mid", 20003, 1200),
                                            ("tiny", 4099, 300)])
def test_views_equal_copied_slots(name, N, nevents):
    w = synth.WORKLOADS[name]
    rb, a, b, grads, slots, (th0_np, grads_np) = _servers(w, N, w.lam + 1)
    ev = rb.Scheduler(w.lam, w.n, w.mode, 23, w.lognormal_sigma, False).next(nevents)
    oracles = []
    for strict in (False, True):
        o = ora.OraclePS(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
        o.set_grad_dtype(w.grad_dtype)
        o.set_weights(th0_np)
        o.set_strict(strict)
        oracles.append(o)
    want_at = {0: (th0_np, th0_np)}          # timestamp -> the oracle's weights (double, fp32 evaluation)
    view_ts = {}                             # learner -> timestamp the oracle handed it last
    rng = np.random.default_rng(2)
    pos = 0
    pulled = set()
    while pos < nevents:
        take = int(rng.integers(1, 150))
        batch = ev[pos:pos + take]
        a.run_events(batch, grads, slots)
        b.run_events(batch, grads, None)
        pos += take
        for e in batch:
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == rb.EV_PUSH:
                for o in oracles:
                    assert o.push(grads_np[l], int(e["pulled_ts"])) > 0
            elif kind == rb.EV_STEP:
                for o in oracles:
                    assert o.step() == 1
                want_at[oracles[0].timestamp()] = (oracles[0].pull()[0], oracles[1].pull()[0])
            elif kind == rb.EV_PULL:
                pulled.add(l)
                view_ts[l] = oracles[0].timestamp()
            elif kind == rb.EV_BROADCAST:
                pulled |= set(range(w.lam))
                view_ts.update({k: oracles[0].timestamp() for k in range(w.lam)})
        a.sync(), b.sync()
        seen = {}
        for l in sorted(pulled):
            ptr, ts = b.view_of(l)
            assert ts == view_ts[l]                         # the version the oracle's learner holds
            if ts not in seen:                              # learners share the buffer: check its contents once
                got = to_host(_view_tensor(ptr, N))
                want, want_fp32 = want_at[ts]
                assert rel_err(got, want) <= REL_100_STEPS
                np.testing.assert_array_equal(got, want_fp32)
            np.testing.assert_array_equal(to_host(_view_tensor(ptr, N)), to_host(slots[l]))
            assert seen.setdefault(ts, ptr) == ptr          # one buffer per timestamp: learners share it
        live = set(view_ts.values()) | {oracles[0].timestamp()}
        want_at = {t: v for t, v in want_at.items() if t in live}
    ca, cb = a.counters(), b.counters()
    assert ca["pulls"] == cb["pulls"] and ca["updates"] == cb["updates"]
    assert cb["weight_copies"] == cb["versions"] <= cb["updates"] + 1
    assert cb["weight_copies"] <= ca["weight_copies"]
    ta, tb = np.empty(N, np.float32), np.empty(N, np.float32)
    a.pull_host(ta), b.pull_host(tb)
    a.sync(), b.sync()
    np.testing.assert_array_equal(ta, tb)
    a.close(), b.close()


def test_a_view_does_not_change_until_its_holder_pulls_again():
    w = synth.WORKLOADS["imagenet"]
    N = 20011
    rb, a, b, grads, slots, _ = _servers(w, N, w.lam + 1)
    ptr, ts = b.pull_view(7)
    assert ts == 0
    before = to_host(_view_tensor(ptr, N)).copy()
    ev = rb.Scheduler(w.lam, w.n, w.mode, 5).next(2000)
    keep = ev[~((ev["learner"] == 7) & (ev["kind"] == rb.EV_PULL))]      # learner 7 never pulls again
    assert b.run_events(keep, grads, None) > 100
    b.sync()
    np.testing.assert_array_equal(to_host(_view_tensor(ptr, N)), before)
    assert b.view_of(7) == (ptr, 0)
    ptr2, ts2 = b.pull_view(7)
    assert ts2 == b.timestamp() and ts2 > 100
    a.close(), b.close()


def test_pool_exhaustion_is_refused_without_side_effects():
    w = synth.WORKLOADS["imagenet"]
    N = 5003
    rb, a, b, grads, slots, _ = _servers(w, N, 3)
    ev = rb.Scheduler(w.lam, w.n, w.mode, 5).next(600)
    before = (b.timestamp(), b.counters())
    with pytest.raises(rb.RudraError) as e:
        b.run_events(ev, grads, None)            # 54 learners at ~18 distinct timestamps need more than 3 versions
    assert e.value.code == rb.E_STATE and "versions" in str(e.value)
    assert (b.timestamp(), b.counters()) == before
    with pytest.raises(rb.RudraError):
        a.pull_view(0)                           # views were never enabled on this handle
    b.enable_views(w.lam + 1)
    assert b.run_events(ev, grads, None) > 0
    with pytest.raises(rb.RudraError) as e:
        b.enable_views(4)                        # learners hold views
    assert e.value.code == rb.E_STATE
    a.close(), b.close()
