"""The workloads at their full stated sizes and lengths, in the launch configuration the benchmark
times (one distinct gradient buffer and one slot per learner, backlogs handed to
rudra_ps_run_events), against the CPU oracle: for the two 60 965 224-weight workloads a sample of
the weights over the whole run (exact, because weights never interact) and the whole vector over
the first updates; for the 1 M-weight workload a sample over its 2 000 updates; for the
CIFAR10-scale workload every weight over its 10 000 updates."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, REL_ONE_STEP, rel_err, to_host

pytestmark = pytest.mark.gpu


def _sample_indices(N, count, seed):
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([np.arange(64), np.arange(N - 64, N), rng.integers(0, N, count)]))


def _host_view(t, w):
    import torch

    return to_host(t.view(torch.int16)).view(np.uint16) if w.grad_dtype == synth.GRAD_BF16 else to_host(t)


def _batches(rb, sched, w, updates, per_batch, cuts):
    """Event batches holding per_batch updates each (the first holds one; a batch also ends when
    the update count reaches one of `cuts`), cut before the push that opens the next update
    window, until `updates` updates have been handed out."""
    out, cur, steps, total, want = [], [], 0, 0, 1
    while total < updates:
        e = sched.next(1)
        if e[0]["kind"] == rb.EV_PUSH and (steps == want or (steps and total in cuts)):
            out.append(np.concatenate(cur))
            cur, steps = [], 0
            want = min(per_batch, updates - total)
        cur.append(e)
        if e[0]["kind"] == rb.EV_STEP:
            steps += 1
            total += 1
    # the pulls that follow the last update belong to its window
    while True:
        e = sched.next(1)
        if e[0]["kind"] == rb.EV_PUSH:
            break
        cur.append(e)
    out.append(np.concatenate(cur))
    return out


def _run_full_size(w, updates, per_batch, max_window, checkpoints, seed, strict=False, whole=False):
    """strict: the oracle evaluates in fp32, one fused multiply-add per term, and the comparison is
    bit for bit.  whole: every weight is compared instead of a sample."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = w.nparams
    idx = np.arange(N) if whole else _sample_indices(N, 20000, seed)
    idx_d = torch.from_numpy(idx).cuda()
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(w.lam)]
    slots = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(w.lam)]
    th0 = synth.device_initial_weights(N, w.theta_std)
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
    ps.set_weights(th0)
    o = ora.OraclePS(len(idx), w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    o.set_grad_dtype(w.grad_dtype)
    o.set_strict(strict)
    o.set_weights(to_host(th0[idx_d]))
    samples = [_host_view(b[idx_d], w) for b in bufs]
    gtable, stable = rb.pointer_table(bufs), rb.pointer_table(slots)
    sched = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED, w.lognormal_sigma, w.downcast)
    th = torch.empty(N, dtype=torch.float32, device="cuda")
    st = torch.empty(N, dtype=torch.float32, device="cuda")
    done, errs, slot_want = 0, {}, {}
    for batch in _batches(rb, sched, w, updates, per_batch, checkpoints):
        got = ps.run_events(batch, gtable, stable, max_window)
        for e in batch:
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == ora.PUSH:
                assert o.push(samples[l], int(e["pulled_ts"])) > 0
            elif kind == ora.STEP:
                assert o.step() == 1
            elif kind == ora.PULL:
                slot_want[l] = o.pull()[0]
            elif kind == ora.BROADCAST:
                cur = o.pull()[0]
                slot_want = {k: cur for k in range(w.lam)}
        done += got
        assert ps.timestamp() == o.timestamp() == done
        g, oc = ps.last_clock(), o.last_clock()
        np.testing.assert_array_equal(g["sigma"], oc["sigma"])
        np.testing.assert_array_equal(g["pulled_ts"], oc["pulled_ts"])
        np.testing.assert_array_equal(g["scale"].view(np.uint32), oc["scale"].view(np.uint32))
        if done in checkpoints or done == updates:
            ps.export_state(th, st)
            ps.sync()
            tol = 0.0 if strict else REL_ONE_STEP if done == 1 else REL_100_STEPS
            e_th = rel_err(to_host(th[idx_d]), o.pull()[0])
            e_st = rel_err(to_host(st[idx_d]), o.state())
            assert e_th <= tol and e_st <= tol, (done, e_th, e_st)
            errs[done] = (e_th, e_st)
    assert done == updates
    ps.sync()
    for l, want in slot_want.items():                         # each learner's copy: what the oracle handed it last
        assert rel_err(to_host(slots[l][idx_d]), want) <= (0.0 if strict else REL_100_STEPS), l
    launches = ps.counters()["launches"]
    ps.close()
    return errs, launches


def test_imagenet_200_updates_at_full_size():
    # lambda = 54, n = 18 (c = 3), momentum 0.9, decay 5e-4, 200 updates; backlogs of one round (18 updates
    # and their 54 pulls) per call, as the benchmark hands them over
    w = synth.WORKLOADS["imagenet"]
    assert w.updates == 200
    errs, launches = _run_full_size(w, 200, 18, 0, {1, 19, 100}, seed=5)
    assert set(errs) >= {1, 100, 200}
    assert launches <= 1 + (200 + 17) // 18 + 3                # one launch per backlog


def test_stress_100_updates_with_their_broadcasts_at_full_size():
    # bf16 gradients, lambda = 128, n = 4 (c = 32), every update followed by the 128-way down-cast, 100 updates
    w = synth.WORKLOADS["stress"]
    assert w.updates == 100
    errs, launches = _run_full_size(w, 100, 1, 1, {1, 2, 50}, seed=6)
    assert set(errs) >= {1, 100}
    assert launches == 200                                      # update + 128-way copy per window


@pytest.mark.parametrize("strict", [False, True])
def test_cifar10_10000_updates_every_weight(strict):
    # 89 578 weights, lambda = n = 30 (c = 1, the staleness of Fig. 3b), momentum 0.9, decay 4e-3, 10 000
    # updates in backlogs of one round (30 updates and their 30 pulls); the 1e-4 bar, stated for 100
    # updates, is held to the end, and the fp32 evaluation of the oracle is matched bit for bit throughout
    w = synth.WORKLOADS["cifar10"]
    assert w.updates == 10000 and w.nparams == 89578
    errs, launches = _run_full_size(w, 10000, 30, 0, {1, 100, 1000, 5000}, seed=7, strict=strict, whole=True)
    assert set(errs) >= {1, 100, 10000}
    assert launches <= 2 + (10000 + 29) // 30 + 4


def test_mid_2000_updates_with_timed_learners():
    # 1 M weights, lambda = 60, n = 4 (c = 15), learners with lognormal(0, 0.3) compute times, 2 000 updates in
    # backlogs of 4 updates as the benchmark hands them over
    w = synth.WORKLOADS["mid"]
    assert w.updates == 2000 and w.nparams == 1000000
    errs, _ = _run_full_size(w, 2000, 4, 0, {1, 100, 1000}, seed=8)
    assert set(errs) >= {1, 100, 2000}
    errs, _ = _run_full_size(w, 200, 4, 0, {1, 100}, seed=9, strict=True)
    assert errs[200] == (0.0, 0.0)


def test_imagenet_whole_vector_against_the_full_size_oracle():
    """Every one of the 60 965 224 weights, state included, after 1, 2 and 3 updates."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    w = synth.WORKLOADS["imagenet"]
    N = w.nparams
    nbuf = 9
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    host = [to_host(b) for b in bufs]
    th0 = synth.device_initial_weights(N, w.theta_std)
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_weights(th0)
    o = ora.OraclePS(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    o.set_weights(to_host(th0))
    sched = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED)
    th = torch.empty(N, dtype=torch.float32, device="cuda")
    st = torch.empty(N, dtype=torch.float32, device="cuda")
    slot = torch.empty(N, dtype=torch.float32, device="cuda")
    done = 0
    while done < 3:
        e = sched.next(1)[0]
        kind, l = int(e["kind"]), int(e["learner"])
        if kind == rb.EV_PUSH:
            ps.push(bufs[l % nbuf], int(e["pulled_ts"]))
            o.push(host[l % nbuf], int(e["pulled_ts"]))
        elif kind == rb.EV_STEP:
            assert ps.step() == 1 and o.step() == 1
            done += 1
            ps.export_state(th, st)
            ps.sync()
            tol = REL_ONE_STEP if done == 1 else REL_100_STEPS
            assert rel_err(to_host(th), o.pull()[0]) <= tol
            assert rel_err(to_host(st), o.state()) <= tol
        elif kind == rb.EV_PULL:
            assert ps.pull(slot) == int(e["ts"])
    assert ps.pull(slot) == 3
    ps.export_state(th, None)
    ps.sync()
    assert torch.equal(slot, th)                                # a pull is an exact copy
    ps.close()
