"""GPU parity: the CUDA library, called through its C interface, against the CPU oracle on the
same seeded inputs.  Integers (timestamps, staleness, grouping, step-size table bits, copied
weights) must agree exactly; weights and state within the stated relative error:
1e-5 after one update and 1e-4 after 100 updates, relative to max(|w_k|, rms(w))."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import (REL_100_STEPS, REL_ONE_STEP, Pair, adagrad_slack, rel_err, rel_err_beyond, run_workload, to_device,
                     to_host)

pytestmark = pytest.mark.gpu


def test_tiny_config_hardsync_100_updates():
    # 4096 weights, lambda = 4, n = 1 (c = 4), momentum 0, 100 updates, every one checked
    errs = run_workload(synth.WORKLOADS["tiny"], 100, check_every=1)
    assert errs[0][0] == 1 and errs[0][1] <= REL_ONE_STEP
    assert errs[-1][0] == 100 and errs[-1][1] <= REL_100_STEPS


def test_tiny_config_hardsync_fused_broadcast():
    errs = run_workload(synth.WORKLOADS["tiny"], 20, check_every=1, fused_pull=True)
    assert len(errs) == 20


def test_tiny_sizes_as_softsync_rounds_shows_staleness():
    w = synth.WORKLOADS["tiny"]
    w2 = synth.Workload("tiny-soft", w.nparams, w.lam, 1, w.alpha0, 0.0, 0.0, synth.SOFTSYNC_ROUNDS, 50, 0.01, 1e-2)
    run_workload(w2, 50, check_every=5, policy=ora.LR_PER_GRADIENT)


def test_cifar10_config_lambda_softsync():
    # ~90 K weights (N = 89578 leaves a ragged tail), lambda = n = 30 (c = 1), momentum + decay
    errs = run_workload(synth.WORKLOADS["cifar10"], 300, check_every=50)
    assert errs[-1][0] == 300


def test_mid_config_timed_learners():
    # 1 M weights, lambda = 60, n = 4 (c = 15), lognormal compute times
    errs = run_workload(synth.WORKLOADS["mid"], 24, check_every=6)
    assert errs[-1][0] == 24


def test_stress_shape_small_bf16_downcast():
    # bf16 gradients, lambda = 128, n = 4 (c = 32), all 128 copies refreshed after every update
    w = synth.WORKLOADS["stress"]
    run_workload(w, 6, check_every=2, N=70001)
    run_workload(w, 4, check_every=2, N=70001, fused_pull=True)


SIZES = [1, 3, 7, 8, 9, 15, 2047, 2048, 2049, 4096 + 5, 8 * 256 * 3 + 1, 8 * 256 * 2 * 5 + 13, 300007]
# lengths at and above 262 144 weights run the 8-weights-per-thread kernel (ragged tiles and tails),
# shorter ones the one-weight-per-thread kernel for small models
VECTOR_SIZES = [262144, 262144 + 1, 262144 + 7, 262144 + 8 * 64 + 9, 262144 + 8 * 256 * 3 + 5, 300007]
GROUPS = [1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 64, 128]


@pytest.mark.parametrize("dtype", [synth.GRAD_F32, synth.GRAD_BF16])
def test_sizes_and_group_widths(dtype):
    # ragged vector lengths x group widths around every unroll boundary of the kernels
    rng = np.random.default_rng(5)
    for i, c in enumerate(GROUPS):
        for N in (SIZES[i % len(SIZES)], SIZES[(3 * i + 1) % len(SIZES)], VECTOR_SIZES[i % len(VECTOR_SIZES)]):
            pair = Pair(N, c, 1, 0.05, 0.9, 5e-4, dtype, policy=ora.LR_PER_GRADIENT, seed=100 + i)
            for step in range(2):
                for l in range(c):
                    p_ts = int(rng.integers(0, pair.gpu.timestamp() + 1))
                    pair.push(synth.gradient(N, l, step, 1e-2, dtype, seed=i), p_ts)
                assert pair.step() == 1
                pair.compare(REL_ONE_STEP if step == 0 else REL_100_STEPS)
            pair.close()


@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_PER_GRADIENT, ora.LR_GROUP_MEAN])
@pytest.mark.parametrize("momentum,wd", [(0.0, 0.0), (0.9, 0.0), (0.0, 5e-4), (0.9, 5e-4)])
def test_policies_and_optimizer_terms(policy, momentum, wd):
    w = synth.Workload("p", 5000, 12, 3, 0.02, momentum, wd, synth.SOFTSYNC_TIMED, 30, 0.01, 1e-2)
    run_workload(w, 30, check_every=10, policy=policy)


def test_adagrad_parity():
    N, lam, n = 33333, 8, 2
    pair = Pair(N, lam, n, 0.01, 0.0, 5e-4, optimizer=ora.OPT_ADAGRAD)
    slack = np.zeros(N)
    for step in range(12):
        for l in range(4):
            pair.push(synth.gradient(N, l, step, 1e-2), pair.gpu.timestamp())
        assert pair.step() == 1
        # the division by sqrt(h) + eps amplifies the fp32 rounding of the mean gradient where h is tiny
        slack += adagrad_slack(pair.cpu.state(), pair.cpu.last_clock()["abar"], 4, 0.06)
        th, st = pair.weights()
        tol = REL_ONE_STEP if step == 0 else REL_100_STEPS
        assert rel_err_beyond(th, pair.cpu.pull()[0], slack) <= tol
        assert rel_err(st, pair.cpu.state()) <= tol
    # the allowance is a sliver of the distance a weight travels (12 steps of about abar each) for all but a few
    assert np.quantile(slack, 0.99) < 1e-3 * 12 * pair.cpu.last_clock()["abar"]
    pair.close()


@pytest.mark.parametrize("N", [70003, 300011])
@pytest.mark.parametrize("dtype,optimizer", [(synth.GRAD_F32, ora.OPT_MOMENTUM_SGD), (synth.GRAD_BF16, ora.OPT_MOMENTUM_SGD),
                                             (synth.GRAD_F32, ora.OPT_ADAGRAD)])
def test_bit_exact_against_the_fp32_evaluation_of_the_oracle(dtype, optimizer, N):
    # Not the parity bar (that is the double-precision oracle, above) but a sharper net: the kernel
    # has no cross-thread reduction, so with the oracle evaluating the same rule in fp32, one fma
    # per term in arrival order, every weight and state value must agree to the last bit.
    lam, n = 15, 3
    pair = Pair(N, lam, n, 0.03, 0.9 if optimizer == ora.OPT_MOMENTUM_SGD else 0.0, 5e-4, dtype,
                policy=ora.LR_PER_GRADIENT, optimizer=optimizer)
    pair.cpu.set_strict(True)
    rng = np.random.default_rng(8)
    for step in range(6):
        for l in range(5):
            pair.push(synth.gradient(N, l, step, 1e-2, dtype), int(rng.integers(0, pair.gpu.timestamp() + 1)))
        assert pair.step() == 1
        th, st = pair.weights()
        np.testing.assert_array_equal(th.view(np.uint32), pair.cpu.pull()[0].view(np.uint32))
        np.testing.assert_array_equal(st.view(np.uint32), pair.cpu.state().view(np.uint32))
    pair.close()


def test_pull_variants_are_exact_copies():
    import torch

    N = 8 * 256 * 4 * 3 + 5
    pair = Pair(N, 3, 1, 0.1, 0.9, 1e-3)
    for l in range(3):
        pair.push(synth.gradient(N, l, 0, 1e-2), 0)
    dsts = [torch.full((N + 16,), 7.0, device="cuda")[8:8 + N] for _ in range(5)]   # guarded by canaries
    assert pair.step(dsts=dsts[:2]) == 1
    th, _ = pair.weights()
    assert pair.gpu.pull(dsts[2]) == 1
    assert pair.gpu.pull_many(dsts[3:]) == 1
    host = np.empty(N, dtype=np.float32)
    assert pair.gpu.pull_host(host) == 1
    pair.gpu.sync()
    for d in dsts:
        np.testing.assert_array_equal(to_host(d), th)
    np.testing.assert_array_equal(host, th)
    np.testing.assert_array_equal(pair.cpu.pull()[0].shape, th.shape)
    assert rel_err(th, pair.cpu.pull()[0]) <= REL_ONE_STEP
    pair.close()


@pytest.mark.parametrize("N", [100003, 300003])
def test_canaries_around_learner_buffers_survive(N):
    import torch

    pair = Pair(N, 2, 1, 0.1, 0.9, 0.0)
    big = torch.full((N + 64,), -123.0, device="cuda")
    dst = big[32:32 + N]
    for l in range(2):
        pair.push(synth.gradient(N, l, 0, 1e-2), 0)
    assert pair.step(dsts=[dst]) == 1
    pair.gpu.pull_many([dst, dst])
    pair.gpu.sync()
    h = to_host(big)
    assert np.all(h[:32] == -123.0) and np.all(h[32 + N:] == -123.0)
    pair.close()


def test_host_buffer_path_matches_device_path():
    import torch

    N, c = 50001, 3
    a = Pair(N, c, 1, 0.05, 0.9, 5e-4)
    b = Pair(N, c, 1, 0.05, 0.9, 5e-4)
    b.gpu.set_weights_host(np.ascontiguousarray(a.theta0))
    for step in range(3):
        for l in range(c):
            g = synth.gradient(N, l, step, 1e-2)
            a.push(g, a.gpu.timestamp())
            pinned = torch.from_numpy(g).pin_memory()
            assert b.gpu.push_host(pinned, b.gpu.timestamp()) == l + 1
        assert a.step() == 1
        assert b.gpu.step() == 1
        out = torch.empty(N, dtype=torch.float32).pin_memory()
        assert b.gpu.pull_host(out) == step + 1
        b.gpu.sync()
        np.testing.assert_array_equal(out.numpy(), a.weights()[0])
    cnt = b.gpu.counters()
    assert cnt["h2d_bytes"] == 4 * N * (1 + 3 * c) and cnt["d2h_bytes"] == 4 * N * 3
    assert cnt["updates"] == 3 and cnt["launches"] == 6 and cnt["pushes"] == 9   # 3 updates + 3 snapshots
    a.close(), b.close()


def test_error_paths_leave_state_untouched():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = 1024
    ps = rb.ParameterServer(N, 4, 2, 0.1, 0.9, 0.0)
    g = torch.zeros(N + 8, device="cuda")
    with pytest.raises(rb.RudraError) as e:
        ps.push(g, 1)                               # timestamp 1 does not exist yet
    assert e.value.code == rb.E_BAD_TS
    with pytest.raises(rb.RudraError) as e:
        ps.push(g[1:], 0)                           # 4-byte offset: not 32-byte aligned
    assert e.value.code == rb.E_INVAL
    with pytest.raises(rb.RudraError) as e:
        ps.push(0, 0)
    assert e.value.code == rb.E_INVAL
    assert ps.step() == 0 and ps.timestamp() == 0   # no gradients: not ready
    assert ps.push(g, 0) == 1
    assert ps.step() == 0 and ps.timestamp() == 0   # one of two: still not ready
    with pytest.raises(rb.RudraError) as e:
        ps.set_option(rb.OPT_LR_POLICY, rb.LR_PER_GRADIENT)
    assert e.value.code == rb.E_STATE
    with pytest.raises(rb.RudraError) as e:
        ps.step_pull_many([g[1:]])
    assert e.value.code == rb.E_INVAL
    assert ps.last_clock()["c"] == 0
    assert ps.push(g, 0) == 2
    assert ps.step() == 1 and ps.timestamp() == 1
    with pytest.raises(rb.RudraError):
        ps.set_option(99, 0)
    ps.sync()
    ps.close()


def test_checkpoint_roundtrip_and_alpha_schedule():
    import torch

    N = 4099
    a = Pair(N, 2, 2, 0.1, 0.9, 1e-3)
    for step in range(3):
        a.push(synth.gradient(N, 0, step, 1e-2), a.gpu.timestamp())
        a.step()
    th = torch.empty(N, device="cuda")
    st = torch.empty(N, device="cuda")
    a.gpu.export_state(th, st)
    from paper_1509_04210_b200 import binding as rb

    b = rb.ParameterServer(N, 2, 2, 0.1, 0.9, 1e-3)
    b.import_state(th, st, 3)
    assert b.timestamp() == 3
    # the step schedule of Section 4.2: rate divided by 10
    for ps in (a.gpu, b):
        ps.set_alpha0(0.01)
    a.cpu.set_alpha0(0.01)
    g = synth.gradient(N, 0, 9, 1e-2)
    gd = to_device(g)
    a.push(g, 2)
    b.push(gd, 2)
    a.step()
    assert b.step() == 1
    th2 = torch.empty(N, device="cuda")
    b.export_state(th2, None)
    b.sync()
    np.testing.assert_array_equal(to_host(th2), a.weights()[0])
    a.compare(REL_100_STEPS)
    a.close(), b.close()


def _sampled_full_size(w, updates, nsample, fused):
    """Full-size run in the benchmark's launch configuration (device-generated buffers, one per
    learner, re-used across that learner's pushes); the oracle recomputes a sample of the weights
    one by one -- exact, because weights never interact."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = w.nparams
    rng = np.random.default_rng(11)
    idx = np.unique(np.concatenate([np.arange(64), np.arange(N - 64, N), rng.integers(0, N, nsample)]))
    idx_d = torch.from_numpy(idx).cuda()
    nbuf = min(w.lam, 2 * w.c + 3)
    bufs = [synth.device_gradient(N, l, w.grad_std, w.grad_dtype) for l in range(nbuf)]
    th0 = synth.device_initial_weights(N, w.theta_std)
    ps = rb.ParameterServer(N, w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    ps.set_option(rb.OPT_GRAD_DTYPE, w.grad_dtype)
    ps.set_weights(th0)
    oc = ora.OraclePS(len(idx), w.lam, w.n, w.alpha0, w.momentum, w.weight_decay)
    oc.set_grad_dtype(w.grad_dtype)
    oc.set_weights(to_host(th0[idx_d]))

    def sample(buf):
        s = buf[idx_d]
        return to_host(s.view(torch.int16)).view(np.uint16) if w.grad_dtype == synth.GRAD_BF16 else to_host(s)

    samples = [sample(b) for b in bufs]
    nslots = 3 if fused else 1
    slots = [torch.empty(N, dtype=torch.float32, device="cuda") for _ in range(nslots)]
    sched = rb.Scheduler(w.lam, w.n, w.mode, synth.MASTER_SEED, w.lognormal_sigma, w.downcast)
    done = 0
    while done < updates:
        ev = sched.next(1)[0]
        if ev["kind"] == rb.EV_PUSH:
            b = int(ev["learner"]) % nbuf
            ps.push(bufs[b], int(ev["pulled_ts"]))
            oc.push(samples[b], int(ev["pulled_ts"]))
        elif ev["kind"] == rb.EV_STEP:
            assert (ps.step_pull_many(slots) if fused else ps.step()) == 1
            assert oc.step() == 1
            done += 1
            g, o = ps.last_clock(), oc.last_clock()
            np.testing.assert_array_equal(g["sigma"], o["sigma"])
            np.testing.assert_array_equal(g["scale"].view(np.uint32), o["scale"].view(np.uint32))
            th = torch.empty(N, dtype=torch.float32, device="cuda")
            st = torch.empty(N, dtype=torch.float32, device="cuda")
            ps.export_state(th, st)
            ps.sync()
            tol = REL_ONE_STEP if done == 1 else REL_100_STEPS
            assert rel_err(to_host(th[idx_d]), oc.pull()[0]) <= tol
            assert rel_err(to_host(st[idx_d]), oc.state()) <= tol
            if fused:
                for s in slots:
                    assert torch.equal(s, th)
        elif ev["kind"] == rb.EV_PULL and not fused:
            assert ps.pull(slots[0]) == int(ev["ts"])
            th = torch.empty(N, dtype=torch.float32, device="cuda")
            ps.export_state(th, None)
            ps.sync()
            assert torch.equal(slots[0], th)
    ps.close()


def test_imagenet_config_full_size_sampled():
    # 60 965 224 weights, lambda = 54, n = 18 (c = 3), momentum 0.9, decay 5e-4
    _sampled_full_size(synth.WORKLOADS["imagenet"], 6, 20000, fused=False)


def test_imagenet_config_full_size_sampled_fused_pulls():
    _sampled_full_size(synth.WORKLOADS["imagenet"], 4, 20000, fused=True)


def test_stress_config_full_size_sampled():
    # 60 965 224 weights, bf16 gradients, lambda = 128, n = 4 (c = 32)
    _sampled_full_size(synth.WORKLOADS["stress"], 3, 20000, fused=True)


def test_floor_group_size_lambda_30_n_4():
    # the paper's own n = 4, lambda = 30 run (Section 5.1): c = floor(30 / 4) = 7
    w = synth.Workload("l30n4", 12345, 30, 4, 0.01, 0.9, 5e-4, synth.SOFTSYNC_ROUNDS, 20, 0.01, 1e-2)
    assert w.c == 7
    run_workload(w, 20, check_every=5)
    run_workload(w, 20, check_every=5, policy=ora.LR_GROUP_MEAN)


def test_single_learner_is_plain_sgd_with_zero_staleness():
    # lambda = 1: n-softsync degenerates to hardsync (Section 5.2); every sigma is 0
    w = synth.Workload("l1", 3001, 1, 1, 0.05, 0.0, 0.0, synth.SOFTSYNC_ROUNDS, 10, 0.01, 1e-2)
    errs = run_workload(w, 10, check_every=1, policy=ora.LR_PER_GRADIENT)
    assert len(errs) == 10


def test_two_handles_on_their_own_streams_do_not_interfere():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = 200003
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    a = Pair(N, 4, 2, 0.05, 0.9, 5e-4, seed=1)
    b = Pair(N, 6, 2, 0.02, 0.0, 1e-3, dtype=synth.GRAD_BF16, seed=2)
    torch.cuda.synchronize()
    a.gpu.set_stream(s1)
    b.gpu.set_stream(s2)
    for step in range(5):
        for l in range(3):                       # interleave the two servers' messages
            if l < 2:
                a.push(synth.gradient(N, l, step, 1e-2, seed=1), a.gpu.timestamp())
            b.push(synth.gradient(N, l, step, 1e-2, synth.GRAD_BF16, seed=2), b.gpu.timestamp())
        assert a.gpu.step() == 1 and b.gpu.step() == 1
        assert a.cpu.step() == 1 and b.cpu.step() == 1
    a.gpu.sync(), b.gpu.sync()
    a._alive.clear(), b._alive.clear()
    a.compare(REL_100_STEPS)
    b.compare(REL_100_STEPS)
    a.close(), b.close()


def test_queue_capacity_is_reported():
    import torch
    from paper_1509_04210_b200 import binding as rb

    ps = rb.ParameterServer(64, 128, 1, 0.1)     # c = 128: nothing steps while we fill the queue
    g = torch.zeros(64, device="cuda")
    for i in range(rb.QUEUE_CAP):
        assert ps.push(g, 0) == i + 1
    with pytest.raises(rb.RudraError) as e:
        ps.push(g, 0)
    assert e.value.code == rb.E_QUEUE_FULL
    done = 0
    while ps.step() == 1:
        done += 1
    assert done == rb.QUEUE_CAP // 128 and ps.timestamp() == done
    ps.close()


def test_a_learner_that_never_pushes():
    # n-softsync needs any c gradients (Eq. 5), so the server keeps advancing without learner 3;
    # hardsync (c = lambda) waits, and the wait is a return value, never a device-side wait.
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = 4096
    g = [to_device(synth.gradient(N, l, 0, 1e-2)) for l in range(4)]
    soft = rb.ParameterServer(N, 4, 2, 0.1)            # c = 2
    for k in range(9):
        soft.push(g[k % 3], soft.timestamp())          # learners 0, 1, 2 only
        assert soft.step() == (1 if k % 2 else 0)
    assert soft.timestamp() == 4
    hard = rb.ParameterServer(N, 4, 1, 0.1)            # c = 4
    for l in range(3):
        hard.push(g[l], 0)
    for _ in range(5):
        assert hard.step() == 0 and hard.timestamp() == 0
    hard.sync()                                        # returns at once: nothing was launched
    assert hard.counters()["launches"] == 0
    hard.push(g[3], 0)
    assert hard.step() == 1
    soft.close(), hard.close()


@pytest.mark.parametrize("optimizer", [ora.OPT_MOMENTUM_SGD, ora.OPT_ADAGRAD])
def test_zero_rate_moves_no_weight(optimizer):
    # alpha0 = 0: every step size is 0 (Eq. 6); the weights stay bit for bit, nothing becomes NaN
    N = 300011
    pair = Pair(N, 3, 1, 0.0, 0.9 if optimizer == ora.OPT_MOMENTUM_SGD else 0.0, 5e-4, optimizer=optimizer)
    for k in range(2):
        for l in range(3):
            pair.push(synth.gradient(N, l, k, 1e-2), pair.gpu.timestamp())
        assert pair.step() == 1
    th, st = pair.weights()
    np.testing.assert_array_equal(th, pair.theta0)
    assert np.isfinite(st).all()
    pair.compare(REL_ONE_STEP)
    pair.close()


def test_one_very_late_gradient_does_not_grow_the_histogram():
    from paper_1509_04210_b200 import binding as rb

    N = 64
    ps = rb.ParameterServer(N, 1, 1, 0.01)
    g = to_device(synth.gradient(N, 0, 0))
    th = to_device(synth.initial_weights(N))
    ps.import_state(th, None, 10**9)               # a server that has been running for a long time
    ps.push(g, 0)                                   # a gradient from the very first weights
    assert ps.step() == 1
    ps.push(g, 10**9 + 1)
    assert ps.step() == 1
    hist = ps.staleness_histogram()
    assert len(hist) == rb.HIST_BINS and hist[-1] == 1 and hist[0] == 1 and hist.sum() == 2
    assert ps.last_clock()["sigma"][0] == 0
    ps.close()


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_mixed_message_kinds_in_one_stream(seed):
    """Every way a gradient can arrive, mixed at random inside the same groups: borrowed device
    buffers, device buffers copied at push time, host buffers uploaded on the side stream; pulls to
    device slots and to host memory in between.  Weights and state must equal the oracle's fp32
    evaluation bit for bit after every update, and be within the bar of its double evaluation."""
    import torch
    from paper_1509_04210_b200 import binding as rb

    rng = np.random.default_rng(1000 + seed)
    N = int(rng.choice([70001, 262144 + 9, 1000003]))
    lam, n = [(6, 2), (8, 2), (12, 4), (5, 1)][seed - 1]
    c = lam // n
    th0 = synth.initial_weights(N, 0.01, seed)
    gpu = rb.ParameterServer(N, lam, n, 0.03, 0.9, 5e-4)
    gpu.set_option(rb.OPT_LR_POLICY, rb.LR_PER_GRADIENT)
    gpu.set_weights(to_device(th0))
    cpus = []
    for strict in (False, True):
        o = ora.OraclePS(N, lam, n, 0.03, 0.9, 5e-4)
        o.set_policy(ora.LR_PER_GRADIENT)
        o.set_strict(strict)
        o.set_weights(th0)
        cpus.append(o)
    th = torch.empty(N, device="cuda")
    st = torch.empty(N, device="cuda")
    slot = torch.empty(N, device="cuda")
    host_dst = torch.empty(N).pin_memory()
    scratch = torch.empty(N, device="cuda")
    keep = []
    for upd in range(1, 9):
        copy_mode = bool(rng.integers(0, 2))                  # the push mode may only change between groups
        gpu.set_option(rb.OPT_PUSH_MODE, rb.PUSH_COPY if copy_mode else rb.PUSH_BORROW)
        for l in range(c):
            g = synth.gradient(N, l, upd, 1e-2, seed=seed)
            p = int(rng.integers(max(0, upd - 3), upd))        # staleness 0, 1 or 2
            if rng.integers(0, 2):
                pinned = torch.from_numpy(g).pin_memory()
                keep.append(pinned)
                gpu.push_host(pinned, p)
            elif copy_mode:
                scratch.copy_(to_device(g))
                gpu.push(scratch, p)
                scratch.fill_(float("nan"))
            else:
                d = to_device(g)
                keep.append(d)
                gpu.push(d, p)
            for o in cpus:
                o.push(g, p)
            if rng.integers(0, 3) == 0:                        # a pull while the group is open
                assert gpu.pull(slot) == upd - 1
        if rng.integers(0, 2):
            assert gpu.step_pull_many([slot]) == 1
        else:
            assert gpu.step() == 1
            if rng.integers(0, 2):
                assert gpu.pull_host(host_dst) == upd
        for o in cpus:
            assert o.step() == 1
        gpu.export_state(th, st)
        gpu.sync()
        g_clock, o_clock = gpu.last_clock(), cpus[0].last_clock()
        np.testing.assert_array_equal(g_clock["sigma"], o_clock["sigma"])
        np.testing.assert_array_equal(g_clock["scale"].view(np.uint32), o_clock["scale"].view(np.uint32))
        np.testing.assert_array_equal(to_host(th), cpus[1].pull()[0])
        np.testing.assert_array_equal(to_host(st), cpus[1].state())
        assert rel_err(to_host(th), cpus[0].pull()[0]) <= (REL_ONE_STEP if upd == 1 else REL_100_STEPS)
    gpu.close()
