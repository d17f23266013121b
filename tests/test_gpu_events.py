"""rudra_ps_run_events (a backlog of messages packed into few launches) against the one-message-at-
a-time calls of the same library -- bit for bit -- and against the CPU oracle within tolerance."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, rel_err, to_device, to_host

pytestmark = pytest.mark.gpu


def _setup(w, N, seed=3):
    import torch
    from paper_1509_04210_b200 import binding as rb

    th0 = synth.initial_weights(N, w.theta_std, seed)
    grads_np = [synth.gradient(N, l, 0, w.grad_std, w.grad_dtype, seed) for l in range(w.lam)]
    grads = [to_device(g) for g in grads_np]

    def make():
        ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
        ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
        ps.set_option(rb.OPT_LR_POLICY, rb.LR_PER_GRADIENT)
        ps.set_weights(to_device(th0))
        slots = [torch.full((N,), float(l), device="cuda") for l in range(w.lam)]
        return ps, slots

    return rb, th0, grads_np, grads, make


def _state(ps, N):
    import torch

    th = torch.empty(N, device="cuda")
    st = torch.empty(N, device="cuda")
    ps.export_state(th, st)
    ps.sync()
    return to_host(th), to_host(st)


def _one_by_one(rb, ps, ev, grads, slots):
    for e in ev:
        k, l = int(e["kind"]), int(e["learner"])
        if k == rb.EV_PUSH:
            ps.push(grads[l], int(e["pulled_ts"]))
        elif k == rb.EV_STEP:
            assert ps.step() == 1
        elif k == rb.EV_PULL:
            assert ps.pull(slots[l]) == int(e["ts"])
        elif k == rb.EV_BROADCAST:
            assert ps.pull_many(slots) == int(e["ts"])


CASES = [
    ("tiny", 4096 + 3, 400, 0),
    ("cifar10", 20011, 700, 0),
    ("mid", 30005, 900, 0),
    ("imagenet", 40001, 1200, 0),
    ("imagenet", 40001, 1200, 5),
    ("imagenet", 300011, 700, 0),
    ("mid", 262144 + 3, 500, 0),
    ("stress", 9001, 1500, 0),
    ("stress", 9001, 1500, 1),
]


EXTRA = {
    # the widest group one launch can carry, with a 128-way broadcast after it
    "hardsync128": synth.Workload("hardsync128", 3001, 128, 1, 0.01, 0.9, 5e-4, synth.HARDSYNC, 0, 0.01, 1e-2),
    # 32 updates of 4 gradients fill the gradient table exactly
    "fill_table": synth.Workload("fill_table", 5003, 128, 32, 0.01, 0.9, 5e-4, synth.SOFTSYNC_TIMED, 0, 0.01, 1e-2),
}
CASES += [("hardsync128", 3001, 800, 0), ("fill_table", 5003, 2500, 0), ("fill_table", 5003, 2500, 7)]


@pytest.mark.parametrize("name,N,nevents,max_window", CASES)
def test_backlog_equals_one_message_at_a_time(name, N, nevents, max_window):
    w = synth.WORKLOADS.get(name) or EXTRA[name]
    rb, th0, grads_np, grads, make = _setup(w, N)
    ev = rb.Scheduler(w.lam, w.n, w.mode, 17, w.lognormal_sigma, w.downcast).next(nevents)
    a, slots_a = make()
    b, slots_b = make()
    _one_by_one(rb, a, ev, grads, slots_a)
    rng = np.random.default_rng(1)
    pos, total = 0, 0
    while pos < nevents:                       # ragged batches: windows start and end anywhere
        take = int(rng.integers(1, 200))
        total += b.run_events(ev[pos:pos + take], grads, slots_b, max_window)
        pos += take
    assert total == int((ev["kind"] == rb.EV_STEP).sum()) == b.timestamp() == a.timestamp()
    tha, sta = _state(a, N)
    thb, stb = _state(b, N)
    np.testing.assert_array_equal(tha, thb)
    if w.momentum:
        np.testing.assert_array_equal(sta, stb)
    for sa, sb in zip(slots_a, slots_b):
        np.testing.assert_array_equal(to_host(sa), to_host(sb))
    ca, cb = a.last_clock(), b.last_clock()
    np.testing.assert_array_equal(ca["sigma"], cb["sigma"])
    np.testing.assert_array_equal(ca["scale"].view(np.uint32), cb["scale"].view(np.uint32))
    assert b.counters()["launches"] < a.counters()["launches"]
    assert b.counters()["pulls"] == a.counters()["pulls"] and b.counters()["updates"] == a.counters()["updates"]
    # and against the oracle
    o = ora.OraclePS(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    o.set_grad_dtype(w.grad_dtype)
    o.set_policy(ora.LR_PER_GRADIENT)
    o.set_weights(th0)
    for e in ev:
        if e["kind"] == ora.PUSH:
            o.push(grads_np[int(e["learner"])], int(e["pulled_ts"]))
        elif e["kind"] == ora.STEP:
            o.step()
    assert rel_err(thb, o.pull()[0]) <= REL_100_STEPS
    if w.momentum:
        assert rel_err(stb, o.state()) <= REL_100_STEPS
    oc = o.last_clock()
    np.testing.assert_array_equal(cb["sigma"], oc["sigma"])
    np.testing.assert_array_equal(cb["pulled_ts"], oc["pulled_ts"])
    a.close(), b.close()


def test_illegal_batch_changes_nothing():
    w = synth.WORKLOADS["imagenet"]
    N = 5000
    rb, th0, grads_np, grads, make = _setup(w, N)
    ps, slots = make()
    ev = rb.Scheduler(w.lam, w.n, w.mode, 17).next(300)
    assert ps.run_events(ev[:100], grads, slots) > 0
    before = (ps.timestamp(), ps.counters(), _state(ps, N)[0].copy())
    bad = ev[100:300].copy()
    k = int(np.flatnonzero(bad["kind"] == rb.EV_PUSH)[-1])
    bad["pulled_ts"][k] = 10**6                                  # a gradient from the future, late in the batch
    with pytest.raises(rb.RudraError) as e:
        ps.run_events(bad, grads, slots)
    assert e.value.code == rb.E_BAD_TS
    bad = ev[100:300].copy()
    bad["ts"][int(np.flatnonzero(bad["kind"] == rb.EV_STEP)[3])] += 1   # trace that does not match the server
    with pytest.raises(rb.RudraError) as e:
        ps.run_events(bad, grads, slots)
    assert e.value.code == rb.E_STATE
    with pytest.raises(rb.RudraError) as e:
        ps.run_events(ev[100:300], grads, None)                  # pulls without slots
    assert e.value.code == rb.E_INVAL
    after = (ps.timestamp(), ps.counters(), _state(ps, N)[0])
    assert before[0] == after[0] and before[1] == after[1]
    np.testing.assert_array_equal(before[2], after[2])
    assert ps.run_events(ev[100:300], grads, slots) > 0          # the legal batch still goes through
    ps.close()


def test_full_size_window_sampled_against_oracle():
    """One round of the 61 M workload (18 updates, 54 pulls) in one launch, the bench's shape;
    the oracle recomputes a sample of the weights."""
    import torch

    w = synth.WORKLOADS["imagenet"]
    N = w.nparams
    from paper_1509_04210_b200 import binding as rb

    rng = np.random.default_rng(3)
    idx = np.unique(np.concatenate([np.arange(64), np.arange(N - 64, N), rng.integers(0, N, 20000)]))
    idx_d = torch.from_numpy(idx).cuda()
    nbuf = 12
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    nslot = 6
    slots = [torch.empty(N, device="cuda") for _ in range(nslot)]
    th0 = synth.device_initial_weights(N, w.theta_std)
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_weights(th0)
    ev = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED).next(54 * 2 + 18 + 54 * 2 + 18)   # two rounds
    assert ps.run_events(ev, [bufs[l % nbuf] for l in range(w.lam)], [slots[l % nslot] for l in range(w.lam)]) == 36
    th = torch.empty(N, device="cuda")
    st = torch.empty(N, device="cuda")
    ps.export_state(th, st)
    ps.sync()
    assert ps.counters()["launches"] <= 4
    o = ora.OraclePS(len(idx), w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    o.set_weights(to_host(th0[idx_d]))
    samples = [to_host(b[idx_d]) for b in bufs]
    last_pull = {}
    for e in ev:
        if e["kind"] == ora.PUSH:
            o.push(samples[int(e["learner"]) % nbuf], int(e["pulled_ts"]))
        elif e["kind"] == ora.STEP:
            o.step()
        elif e["kind"] == ora.PULL:
            last_pull[int(e["learner"]) % nslot] = o.pull()[0]
    assert rel_err(to_host(th[idx_d]), o.pull()[0]) <= REL_100_STEPS
    assert rel_err(to_host(st[idx_d]), o.state()) <= REL_100_STEPS
    for s, want in last_pull.items():                            # the last writer of each slot wins
        assert rel_err(to_host(slots[s][idx_d]), want) <= REL_100_STEPS
    ps.close()


@pytest.mark.parametrize("dtype", [synth.GRAD_F32, synth.GRAD_BF16])
def test_broadcast_dominated_launch_equals_update_then_copies(dtype):
    """An update that also serves 64 learner buffers is split by the library into the update and
    a 64-way copy when the vector is large; either way it must equal the two explicit calls."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, lam, n = 5000011, 64, 2
    c = lam // n
    th0 = synth.device_initial_weights(N, 0.01)
    grads = [synth.device_gradient(N, l, 1e-3, dtype) for l in range(c)]
    out = []
    for fused in (False, True):
        ps = rb.ParameterServer(N, lam, n, 0.01, 0.9, 5e-4)
        ps.set_option(rb.OPT_GRAD_DTYPE, dtype)
        ps.set_weights(th0)
        slots = [torch.full((N,), 3.0, device="cuda") for _ in range(lam)]
        for step in range(2):
            for l in range(c):
                ps.push(grads[(l + step) % c], max(0, ps.timestamp() - (l % 2)))
            if fused:
                assert ps.step_pull_many(slots) == 1
            else:
                assert ps.step() == 1
                assert ps.pull_many(slots) == ps.timestamp()
        th = torch.empty(N, device="cuda")
        st = torch.empty(N, device="cuda")
        ps.export_state(th, st)
        ps.sync()
        out.append((th, st, slots))
        ps.close()
    (tha, sta, sa), (thb, stb, sb) = out
    assert torch.equal(tha, thb) and torch.equal(sta, stb)
    for i in (0, 1, 31, 63):
        assert torch.equal(sa[i], tha) and torch.equal(sb[i], thb)


def test_stress_config_full_size_backlog_sampled_against_oracle():
    """The bf16, c = 32, 128-way down-cast workload at 60 965 224 weights, driven as the bench
    drives it (one update and its broadcast per run_events call); the oracle recomputes a sample."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    w = synth.WORKLOADS["stress"]
    N = w.nparams
    rng = np.random.default_rng(4)
    idx = np.unique(np.concatenate([np.arange(64), np.arange(N - 64, N), rng.integers(0, N, 20000)]))
    idx_d = torch.from_numpy(idx).cuda()
    nbuf = 40
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    slots = [torch.empty(N, device="cuda") for _ in range(w.lam)]
    th0 = synth.device_initial_weights(N, w.theta_std)
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
    ps.set_weights(th0)
    o = ora.OraclePS(len(idx), w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    o.set_grad_dtype(w.grad_dtype)
    o.set_weights(to_host(th0[idx_d]))
    samples = [to_host(b[idx_d].view(torch.int16)).view(np.uint16) for b in bufs]
    sched = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED, w.lognormal_sigma, w.downcast)
    gt = [bufs[l % nbuf] for l in range(w.lam)]
    updates = 0
    while updates < 3:
        ev = sched.next(1)
        batch = [ev]
        while ev[0]["kind"] != rb.EV_BROADCAST:       # one update window: 32 pushes, the update, the broadcast
            ev = sched.next(1)
            batch.append(ev)
        batch = np.concatenate(batch)
        assert ps.run_events(batch, gt, slots, 1) == 1
        for e in batch:
            if e["kind"] == ora.PUSH:
                o.push(samples[int(e["learner"]) % nbuf], int(e["pulled_ts"]))
            elif e["kind"] == ora.STEP:
                assert o.step() == 1
        updates += 1
        th = torch.empty(N, device="cuda")
        st = torch.empty(N, device="cuda")
        ps.export_state(th, st)
        ps.sync()
        tol = 1e-5 if updates == 1 else REL_100_STEPS
        assert rel_err(to_host(th[idx_d]), o.pull()[0]) <= tol
        assert rel_err(to_host(st[idx_d]), o.state()) <= tol
        np.testing.assert_array_equal(ps.last_clock()["sigma"], o.last_clock()["sigma"])
        for i in (0, 63, 127):
            assert torch.equal(slots[i], th)           # every learner received this version
    assert ps.counters()["launches"] == 6             # update + 128-way copy per window
    ps.close()


def test_clock_log_and_staleness_histogram_match_the_trace():
    """The server's record of its updates (vector clock per update, <sigma> of Eq. 2, staleness
    histogram: the data behind the paper's Fig. 3) against the oracle and the event trace."""
    from paper_1509_04210_b200 import binding as rb

    lam, n, N = 30, 30, 2048                       # the lambda-softsync case of Section 5.1
    w = synth.Workload("fig3b", N, lam, n, 0.001, 0.9, 0.0, synth.SOFTSYNC_ROUNDS, 0, 0.01, 1e-3)
    rb_, th0, grads_np, grads, make = _setup(w, N)
    ps, slots = make()
    ev = rb.Scheduler(lam, n, w.mode, 3).next(9000)
    pos = 0
    while pos < len(ev):
        ps.run_events(ev[pos:pos + 700], grads, slots)
        pos += 700
    ps.sync()
    pushes = ev[ev["kind"] == rb.EV_PUSH]
    K = ps.timestamp()
    assert K == len(pushes) == 3000                # c = 1: every push is an update
    pulled, avg = ps.clock_log(0, K)
    assert len(avg) == K
    np.testing.assert_array_equal(pulled[:, 0], pushes["pulled_ts"])
    sigma = (pushes["ts"] - pushes["pulled_ts"]).astype(np.int64)
    np.testing.assert_array_equal(avg, sigma.astype(np.float64))          # Eq. 2 with c = 1
    hist = ps.staleness_histogram()
    np.testing.assert_array_equal(hist, np.bincount(sigma, minlength=len(hist)))
    assert abs(sigma[2 * lam:].mean() - 29.0) < 0.5 and sigma.max() <= 2 * n   # <sigma> close to 30, at most 2n
    # a grouped case against the oracle's per-update records
    w2 = synth.WORKLOADS["imagenet"]
    rb_, th0, grads_np, grads, make = _setup(w2, 1024)
    ps2, slots2 = make()
    o = ora.OraclePS(1024, w2.lam, w2.n, w2.alpha0, w2.momentum, w2.weight_decay)
    o.set_weights(th0)
    ev = rb.Scheduler(w2.lam, w2.n, w2.mode, 3).next(2000)
    ps2.run_events(ev, grads, slots2)
    want_p, want_a = [], []
    for e in ev:
        if e["kind"] == ora.PUSH:
            o.push(grads_np[int(e["learner"])], int(e["pulled_ts"]))
        elif e["kind"] == ora.STEP:
            o.step()
            rec = o.last_clock()
            want_p.append(rec["pulled_ts"].copy())
            want_a.append(rec["avg_sigma"])
    pulled, avg = ps2.clock_log(0, 10 ** 6)
    np.testing.assert_array_equal(pulled, np.array(want_p))
    np.testing.assert_array_equal(avg, np.array(want_a))
    late, _ = ps2.clock_log(len(want_a) - 5, 100)
    np.testing.assert_array_equal(late, np.array(want_p[-5:]))
    ps.close(), ps2.close()
