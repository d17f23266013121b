"""The two-level server tree of Section 3.3 (Rudra-adv) through the C interface, against the CPU
oracle: the leaf's averaging kernel, relayed averages at the root, raw groups averaged inside the
update kernel, and whole event streams of learners -> leaves -> root."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, REL_ONE_STEP, adagrad_slack, rel_err, rel_err_beyond, to_device, to_host

pytestmark = pytest.mark.gpu


def _grad(N, l, seq, dtype, seed=31):
    return synth.gradient(N, l, seq, 1e-2, dtype, seed)


@pytest.mark.parametrize("dtype", [synth.GRAD_F32, synth.GRAD_BF16])
@pytest.mark.parametrize("N,k", [(1, 1), (7, 3), (4096, 4), (100003, 5), (300011, 8), (300011, 33)])
def test_leaf_average_kernel(N, k, dtype):
    """The leaf's kernel alone: the fp32 fused-multiply-add chain bit for bit, the exact mean within
    one rounding per term, and nothing written outside the output."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    gs = [_grad(N, l, 0, dtype) for l in range(k)]
    dev = [to_device(g) for g in gs]
    big = torch.full((N + 16,), -7.0, device="cuda")
    out = big[8:8 + N]
    assert rb.leaf_average(dev, dtype, N, out) == 0
    torch.cuda.synchronize()
    wide = [synth.bf16_bits_to_f32(g) if dtype == synth.GRAD_BF16 else g for g in gs]
    inv_k = np.float32(1.0 / k)
    # fma(inv_k, g, acc) has one rounding: evaluate it in double (the product of two floats is exact
    # there and the sum of it with a float rounds to double first, but stays within half an fp32 ulp of
    # the fused result except in rare double-rounding cases) and allow that one ulp
    acc = np.zeros(N, dtype=np.float32)
    for g in wide:
        acc = (inv_k.astype(np.float64) * g.astype(np.float64) + acc.astype(np.float64)).astype(np.float32)
    got = to_host(out)
    assert np.max(np.abs(got.view(np.int32).astype(np.int64) - acc.view(np.int32).astype(np.int64))) <= 1
    mean = np.mean(np.stack(wide).astype(np.float64), axis=0)
    assert np.max(np.abs(got - mean)) <= (k + 1) * np.finfo(np.float32).eps * np.max(np.abs(np.stack(wide)))
    h = to_host(big)
    assert np.all(h[:8] == -7.0) and np.all(h[8 + N:] == -7.0)


def _pair(N, lam, n, policy, opt, m, wd, dtype=synth.GRAD_F32, a0=0.05, seed=9):
    from paper_1509_04210_b200 import binding as rb

    th0 = synth.initial_weights(N, 0.01, seed)
    gpu = rb.ParameterServer(N, lam, n, a0, m, wd)
    gpu.set_option(rb.OPT_GRAD_DTYPE, dtype)
    gpu.set_option(rb.OPT_LR_POLICY, policy)
    gpu.set_option(rb.OPT_OPTIMIZER, opt)
    gpu.set_weights(to_device(th0))
    cpus = []
    for strict in (False, True):
        o = ora.OraclePS(N, lam, n, a0, m, wd)
        o.set_grad_dtype(dtype)
        o.set_policy(policy)
        o.set_optimizer(opt, 1e-8)
        o.set_weights(th0)
        o.set_strict(strict)
        cpus.append(o)
    return rb, gpu, cpus


def _state(gpu, N):
    import torch

    th, st = torch.empty(N, device="cuda"), torch.empty(N, device="cuda")
    gpu.export_state(th, st)
    gpu.sync()
    return to_host(th), to_host(st)


def _check_integers(gpu, cpu):
    g, o = gpu.last_clock(), cpu.last_clock()
    np.testing.assert_array_equal(g["pulled_ts"], o["pulled_ts"])
    np.testing.assert_array_equal(g["sigma"], o["sigma"])
    np.testing.assert_array_equal(g["scale"].view(np.uint32), o["scale"].view(np.uint32))
    assert g["avg_sigma"] == o["avg_sigma"]
    gm, om = gpu.last_messages(), cpu.last_messages()
    np.testing.assert_array_equal(gm["fanin"], om["fanin"])
    np.testing.assert_array_equal(gm["step"].view(np.uint32), om["step"].view(np.uint32))
    assert gpu.timestamp() == cpu.timestamp()


@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_PER_GRADIENT, ora.LR_GROUP_MEAN])
@pytest.mark.parametrize("opt,m", [(ora.OPT_MOMENTUM_SGD, 0.9), (ora.OPT_MOMENTUM_SGD, 0.0), (ora.OPT_ADAGRAD, 0.0)])
@pytest.mark.parametrize("N,leaf_dtype", [(70003, synth.GRAD_F32), (300011, synth.GRAD_F32), (300011, synth.GRAD_BF16)])
def test_relayed_averages_at_the_root(N, leaf_dtype, opt, m, policy):
    """Leaves run rudra_leaf_average and relay one float vector each (rudra_ps_push_group with
    nvec = 1); the root must do what the oracle's root does with the oracle's leaf averages:
    integers and step sizes bit for bit, weights within tolerance of the double evaluation and bit
    for bit the fp32 evaluation.  lambda = 12, n = 2: c = 6 as 2 leaves of 3."""
    import torch

    lam, n, k = 12, 2, 3
    rb, gpu, cpus = _pair(N, lam, n, policy, opt, m, 5e-4)
    for o in cpus:
        o.set_grad_dtype(leaf_dtype)         # what the leaves receive; the root receives float averages
    avgs = [torch.empty(N, device="cuda") for _ in range(2)]
    slack = np.zeros(N)
    for upd in range(5):
        ts = gpu.timestamp()
        for leaf in range(2):
            gs = [_grad(N, leaf * k + i, upd, leaf_dtype) for i in range(k)]
            stamps = [max(0, ts - ((leaf + i + upd) % 4)) for i in range(k)]
            dev = [to_device(g) for g in gs]
            assert rb.leaf_average(dev, leaf_dtype, N, avgs[leaf]) == 0
            want_q = gpu.push_group([avgs[leaf]], stamps)
            for o in cpus:
                assert o.push_relay(gs, stamps) == want_q
        assert gpu.step() == 1
        gpu.sync()
        for o in cpus:
            assert o.step() == 1
        _check_integers(gpu, cpus[0])
        th, st = _state(gpu, N)
        tol = REL_ONE_STEP if upd == 0 else REL_100_STEPS
        if opt == ora.OPT_ADAGRAD:   # the division by sqrt(h) + eps amplifies fp32 rounding where h is tiny
            slack += adagrad_slack(cpus[0].state(), cpus[0].last_clock()["abar"], 2 * k, 0.06)
        assert rel_err_beyond(th, cpus[0].pull()[0], slack) <= tol
        np.testing.assert_array_equal(th, cpus[1].pull()[0])
        if m or opt == ora.OPT_ADAGRAD:
            assert rel_err(st, cpus[0].state()) <= tol
            np.testing.assert_array_equal(st, cpus[1].state())
    gpu.close()


@pytest.mark.parametrize("dtype", [synth.GRAD_F32, synth.GRAD_BF16])
@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_PER_GRADIENT])
@pytest.mark.parametrize("N", [4099, 300011])
def test_raw_groups_averaged_inside_the_update_kernel(N, policy, dtype):
    """A leaf on the root's GPU hands over its k raw vectors (nvec = k): same integers and step
    sizes; weights within tolerance (the average is not rounded to a float vector on the way, so
    the fp32 evaluation of the oracle is not reproduced bit for bit).  A learner attached to the
    root directly shares the group: c = 7 as leaves of 4 and 2 and one direct push."""
    lam, n = 7, 1
    rb, gpu, cpus = _pair(N, lam, n, policy, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4, dtype)
    cpu = cpus[0]
    for upd in range(4):
        ts = gpu.timestamp()
        gs = [_grad(N, l, upd, dtype) for l in range(7)]
        st = [max(0, ts - (l % 3)) for l in range(7)]
        dev = [to_device(g) for g in gs]
        assert gpu.push_group(dev[0:4], st[0:4]) == cpu.push_relay(gs[0:4], st[0:4]) == 4
        assert gpu.push(dev[4], st[4]) == cpu.push(gs[4], st[4]) == 5
        assert gpu.push_group(dev[5:7], st[5:7]) == cpu.push_relay(gs[5:7], st[5:7]) == 7
        assert gpu.step() == 1 and cpu.step() == 1
        gpu.sync()
        _check_integers(gpu, cpu)
        assert list(gpu.last_messages()["fanin"]) == [4, 1, 2]
        th, stt = _state(gpu, N)
        tol = REL_ONE_STEP if upd == 0 else REL_100_STEPS
        assert rel_err(th, cpu.pull()[0]) <= tol and rel_err(stt, cpu.state()) <= tol
    gpu.close()


TREE_STREAMS = [
    # name, N, lambda, n, fan-in, mode, events
    ("rounds", 30011, 12, 2, 3, synth.SOFTSYNC_ROUNDS, 900),
    ("imagenet-shape", 280003, 54, 18, 3, synth.SOFTSYNC_ROUNDS, 1500),
    ("wide-leaves", 9001, 54, 3, 6, synth.SOFTSYNC_ROUNDS, 1200),
    ("timed", 20003, 60, 4, 5, synth.SOFTSYNC_TIMED, 1500),
    ("hardsync", 4099, 8, 1, 4, synth.HARDSYNC, 400),
]


@pytest.mark.parametrize("name,N,lam,n,k,mode,nevents", TREE_STREAMS)
@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_PER_GRADIENT])
def test_event_stream_through_the_tree(name, N, lam, n, k, mode, nevents, policy):
    """learners -> leaves -> root as rudra_ps_run_events plays it (RUDRA_OPT_TREE_FANIN, ragged
    backlogs), against the oracle fed the same events one by one."""
    import torch

    rb, gpu, cpus = _pair(N, lam, n, policy, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4, a0=0.01)
    cpu = cpus[0]
    gpu.set_option(rb.OPT_TREE_FANIN, k)
    grads_np = [_grad(N, l, 0, synth.GRAD_F32) for l in range(lam)]
    grads = [to_device(g) for g in grads_np]
    slots = [torch.full((N,), -1.0, device="cuda") for _ in range(lam)]
    ev = rb.Scheduler(lam, n, mode, 23, 0.3, False, k).next(nevents)
    assert ev.tobytes() == ora.OracleScheduler(lam, n, mode, 23, 0.3, False, k).run(nevents).tobytes()
    rng = np.random.default_rng(4)
    pos, updates = 0, 0
    at_leaf = {}
    slot_want = {}
    while pos < nevents:
        batch = ev[pos:pos + int(rng.integers(1, 200))]
        pos += len(batch)
        got = gpu.run_events(batch, grads, slots)
        for e in batch:
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == ora.PUSH:
                at_leaf.setdefault(l // k, []).append((grads_np[l], int(e["pulled_ts"])))
            elif kind == ora.RELAY:
                msg = at_leaf.pop(l)
                assert cpu.push_relay([g for g, _ in msg], [p for _, p in msg]) > 0
            elif kind == ora.STEP:
                assert cpu.step() == 1
            elif kind == ora.PULL:
                slot_want[l] = cpu.pull()[0]
            elif kind == ora.BROADCAST:
                cur = cpu.pull()[0]
                slot_want = {j: cur for j in range(lam)}
        updates += got
        assert gpu.timestamp() == cpu.timestamp() == updates
        if got:
            _check_integers(gpu, cpu)
        th, st = _state(gpu, N)
        assert rel_err(th, cpu.pull()[0]) <= REL_100_STEPS and rel_err(st, cpu.state()) <= REL_100_STEPS
    assert updates > 10
    for l, want in slot_want.items():
        assert rel_err(to_host(slots[l]), want) <= REL_100_STEPS
    gpu.close()


def test_tree_at_61m_weights_sampled():
    """The ImageNet-scale vector behind a tree of 18 leaves of 3 learners, one round per call."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    w = synth.WORKLOADS["imagenet"]
    N, k = w.nparams, 3
    rng = np.random.default_rng(8)
    idx = np.unique(np.concatenate([np.arange(64), np.arange(N - 64, N), rng.integers(0, N, 20000)]))
    idx_d = torch.from_numpy(idx).cuda()
    nbuf = 18
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    samples = [to_host(b[idx_d]) for b in bufs]
    slots = [torch.empty(N, device="cuda") for _ in range(6)]
    th0 = synth.device_initial_weights(N, w.theta_std)
    gpu = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    gpu.set_option(rb.OPT_LR_POLICY, rb.LR_PER_GRADIENT)
    gpu.set_option(rb.OPT_TREE_FANIN, k)
    gpu.set_weights(th0)
    cpu = ora.OraclePS(len(idx), w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    cpu.set_policy(ora.LR_PER_GRADIENT)
    cpu.set_weights(to_host(th0[idx_d]))
    sched = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED, 0.3, False, k)
    gt = [bufs[l % nbuf] for l in range(w.lam)]
    stt = [slots[l % 6] for l in range(w.lam)]
    th, st = torch.empty(N, device="cuda"), torch.empty(N, device="cuda")
    at_leaf, updates = {}, 0
    for rnd in range(3):
        batch = sched.next(54 + 18 + 18 + 54)          # one round: pushes, relays, updates, pulls
        updates += gpu.run_events(batch, gt, stt)
        for e in batch:
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == ora.PUSH:
                at_leaf.setdefault(l // k, []).append((samples[l % nbuf], int(e["pulled_ts"])))
            elif kind == ora.RELAY:
                msg = at_leaf.pop(l)
                cpu.push_relay([g for g, _ in msg], [p for _, p in msg])
            elif kind == ora.STEP:
                assert cpu.step() == 1
        assert updates == cpu.timestamp() == 18 * (rnd + 1)
        _check_integers(gpu, cpu)
        gpu.export_state(th, st)
        gpu.sync()
        assert rel_err(to_host(th[idx_d]), cpu.pull()[0]) <= REL_100_STEPS
        assert rel_err(to_host(st[idx_d]), cpu.state()) <= REL_100_STEPS
    assert gpu.counters()["launches"] <= 3 * 2         # 54 raw vectors per round fit one launch's table
    gpu.close()


def test_group_messages_that_do_not_fit_are_refused():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = 1024
    gpu = rb.ParameterServer(N, 6, 2, 0.1)                  # c = 3
    g = [torch.zeros(N, device="cuda") for _ in range(4)]
    assert gpu.push(g[0], 0) == 1 and gpu.push(g[1], 0) == 2
    for vecs, stamps, code in [
        (g[:2], [0, 0], rb.E_STATE),                        # 2 + 2 > c: would straddle two updates
        (g[:4], [0, 0, 0, 0], rb.E_INVAL),                  # more than a whole group
        (g[:1], [1], rb.E_BAD_TS),                          # weights with timestamp 1 do not exist
        (g[:2], [0, 0, 0], rb.E_INVAL),                     # neither one average nor one vector per gradient
        ([g[0][1:]], [0], rb.E_INVAL),                      # misaligned
    ]:
        with pytest.raises(rb.RudraError) as e:
            gpu.push_group(vecs, stamps)
        assert e.value.code == code, (stamps, e.value)
    assert gpu.step() == 0 and gpu.counters()["pushes"] == 2
    assert gpu.push_group(g[:1], [0]) == 3 and gpu.step() == 1
    gpu.set_option(rb.OPT_GRAD_DTYPE, rb.GRAD_BF16)
    with pytest.raises(rb.RudraError) as e:
        gpu.push_group(g[:1], [0, 0])                       # an average is a float vector
    assert e.value.code == rb.E_STATE
    with pytest.raises(rb.RudraError):
        gpu.set_option(rb.OPT_TREE_FANIN, 2)                # 2 does not divide c = 3
    ev = rb.Scheduler(6, 2, rb.SCHED_SOFTSYNC_ROUNDS, 1, 0.3, False, 3).next(50)
    with pytest.raises(rb.RudraError) as e:
        gpu.run_events(ev, g[:4] + g[:2], None)             # RELAY events, but the handle plays no tree
    assert e.value.code == rb.E_STATE
    gpu.close()


def test_copy_push_into_a_slot_whose_upload_was_dropped_unread():
    """Gradients pushed from host memory are still on their way when set_weights drops the queue; the
    COPY-mode pushes that follow reuse those staging slots and must not be overtaken by the uploads."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, lam, n = 1000003, 6, 2
    rb, gpu, cpus = _pair(N, lam, n, ora.LR_PAPER_N, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4)
    cpu = cpus[0]
    junk = [torch.full((N,), 1e30).pin_memory() for _ in range(3)]
    th0 = synth.initial_weights(N, 0.01, 9)
    for rounds in range(3):
        for j in junk:                                        # uploads nobody will read
            gpu.push_host(j, 0)
        gpu.set_weights(to_device(th0))                       # drops them; timestamps start over
        cpu.set_weights(th0)
        gpu.set_option(rb.OPT_PUSH_MODE, rb.PUSH_COPY)
        gs = [_grad(N, l, rounds, synth.GRAD_F32) for l in range(3)]
        scratch = torch.empty(N, device="cuda")
        for g in gs:
            scratch.copy_(to_device(g))
            gpu.push(scratch, 0)
            cpu.push(g, 0)
            scratch.fill_(float("nan"))
        assert gpu.step() == 1 and cpu.step() == 1
        th, _ = _state(gpu, N)
        assert np.isfinite(th).all()
        assert rel_err(th, cpu.pull()[0]) <= REL_ONE_STEP
        gpu.set_option(rb.OPT_PUSH_MODE, rb.PUSH_BORROW)
    gpu.close()


@pytest.mark.parametrize("N", [70003, 300011])
def test_copy_push_mode_lets_the_caller_overwrite_its_buffer(N):
    """Section 3.2's push message carries the gradient: with RUDRA_PUSH_COPY the server owns a copy
    from the moment the push returns.  One caller buffer is overwritten right after every push
    (on the same stream); the result must be the oracle's, and bit for bit that of borrowed buffers."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    lam, n = 6, 2
    rb, a, cpus = _pair(N, lam, n, ora.LR_PER_GRADIENT, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4)
    _, b, _ = _pair(N, lam, n, ora.LR_PER_GRADIENT, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4)
    b.set_option(rb.OPT_PUSH_MODE, rb.PUSH_COPY)
    cpu = cpus[0]
    scratch = torch.empty(N, device="cuda")                  # the only gradient buffer the COPY caller has
    keep = []
    for upd in range(4):
        ts = a.timestamp()
        gs = [_grad(N, l, upd, synth.GRAD_F32) for l in range(3)]
        stamps = [max(0, ts - l) for l in range(3)]
        dev = [to_device(g) for g in gs]
        keep += dev
        if upd % 2 == 0:
            for g, d, p in zip(gs, dev, stamps):
                a.push(d, p)
                cpu.push(g, p)
                scratch.copy_(d)
                b.push(scratch, p)
                scratch.fill_(float("nan"))                  # ordered after the push on the same stream
        else:                                                # the same through group messages
            a.push_group(dev[:2], stamps[:2]), a.push(dev[2], stamps[2])
            cpu.push_relay(gs[:2], stamps[:2]), cpu.push(gs[2], stamps[2])
            two = [d.clone() for d in dev[:2]]
            b.push_group(two, stamps[:2])
            for t in two:
                t.fill_(float("nan"))
            scratch.copy_(dev[2])
            b.push(scratch, stamps[2])
            scratch.fill_(float("nan"))
        assert a.step() == 1 and b.step() == 1 and cpu.step() == 1
        tha, sta = _state(a, N)
        thb, stb = _state(b, N)
        np.testing.assert_array_equal(tha, thb)
        np.testing.assert_array_equal(sta, stb)
        assert np.isfinite(thb).all()
        assert rel_err(thb, cpu.pull()[0]) <= (REL_ONE_STEP if upd == 0 else REL_100_STEPS)
    # and through a backlog of events
    ev = rb.Scheduler(lam, n, rb.SCHED_SOFTSYNC_ROUNDS, 3).next(300)
    base = a.timestamp()
    ev["ts"] += base
    ev["pulled_ts"] += base
    grads = [to_device(_grad(N, l, 99, synth.GRAD_F32)) for l in range(lam)]
    mine = [g.clone() for g in grads]
    slots = [torch.empty(N, device="cuda") for _ in range(lam)]
    na = a.run_events(ev, grads, slots)
    nb = b.run_events(ev, mine, slots)
    for m in mine:
        m.fill_(float("nan"))
    assert na == nb > 20
    tha, sta = _state(a, N)
    thb, stb = _state(b, N)
    np.testing.assert_array_equal(tha, thb)
    np.testing.assert_array_equal(sta, stb)
    a.close(), b.close()


@pytest.mark.parametrize("N", [1, 5, 8, 4099])
def test_widest_tree_group_fills_the_launch_table(N):
    """lambda = 128, n = 1: one update of c = 128 gradients (the table's limit) as two leaves of 64,
    once as raw vectors and once as relayed averages, on vectors shorter than one 256-bit unit too."""
    import torch

    lam, k = 128, 64
    for relayed in (False, True):
        rb, gpu, cpus = _pair(N, lam, 1, ora.LR_PER_GRADIENT, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4)
        cpu = cpus[0]
        for upd in range(2):
            ts = gpu.timestamp()
            keep = []
            for leaf in range(2):
                gs = [_grad(N, leaf * k + i, upd, synth.GRAD_F32) for i in range(k)]
                stamps = [max(0, ts - (i % 2)) for i in range(k)]
                dev = [to_device(g) for g in gs]
                keep.append(dev)
                if relayed:
                    avg = torch.empty(N, device="cuda")
                    keep.append(avg)
                    rb.leaf_average(dev, synth.GRAD_F32, N, avg)
                    gpu.push_group([avg], stamps)
                else:
                    gpu.push_group(dev, stamps)
                cpu.push_relay(gs, stamps)
            assert gpu.step() == 1 and cpu.step() == 1
            gpu.sync()
            _check_integers(gpu, cpu)
            th, st = _state(gpu, N)
            tol = REL_ONE_STEP if upd == 0 else REL_100_STEPS
            assert rel_err(th, cpu.pull()[0]) <= tol and rel_err(st, cpu.state()) <= tol
        gpu.close()


def test_empty_batches_and_partial_leaves_carry_over():
    """run_events with no events does nothing; a leaf left half full at the end of a batch is
    completed by the next batch; options cannot change while a leaf holds a gradient."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, lam, n, k = 3001, 8, 2, 2
    rb, gpu, cpus = _pair(N, lam, n, ora.LR_PAPER_N, ora.OPT_MOMENTUM_SGD, 0.9, 5e-4)
    cpu = cpus[0]
    gpu.set_option(rb.OPT_TREE_FANIN, k)
    grads_np = [_grad(N, l, 0, synth.GRAD_F32) for l in range(lam)]
    grads = [to_device(g) for g in grads_np]
    slots = [torch.empty(N, device="cuda") for _ in range(lam)]
    ev = rb.Scheduler(lam, n, rb.SCHED_SOFTSYNC_ROUNDS, 3, 0.3, False, k).next(200)
    assert gpu.run_events(ev[:0], grads, slots) == 0 and gpu.timestamp() == 0
    first_push = int(np.flatnonzero(ev["kind"] == rb.EV_PUSH)[0])
    assert gpu.run_events(ev[: first_push + 1], grads, slots) == 0          # one gradient sits at its leaf
    with pytest.raises(rb.RudraError) as e:
        gpu.set_option(rb.OPT_LR_POLICY, rb.LR_GROUP_MEAN)
    assert e.value.code == rb.E_STATE
    done = gpu.run_events(ev[first_push + 1:], grads, slots)
    at_leaf = {}
    for e in ev:
        kind, l = int(e["kind"]), int(e["learner"])
        if kind == ora.PUSH:
            at_leaf.setdefault(l // k, []).append((grads_np[l], int(e["pulled_ts"])))
        elif kind == ora.RELAY:
            msg = at_leaf.pop(l)
            cpu.push_relay([g for g, _ in msg], [p for _, p in msg])
        elif kind == ora.STEP:
            assert cpu.step() == 1
    assert done == cpu.timestamp() == gpu.timestamp() > 10
    th, st = _state(gpu, N)
    assert rel_err(th, cpu.pull()[0]) <= REL_100_STEPS and rel_err(st, cpu.state()) <= REL_100_STEPS
    gpu.close()
