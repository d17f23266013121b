"""Seeded random protocol configurations through rudra_ps_run_events against the CPU oracle:
learner counts, splitting parameters, vector lengths around the kernels' tile and unit boundaries,
rate policies, optimizers, gradient types, scheduler modes, server-tree fan-ins, push modes and
ragged backlog sizes drawn together, so that table limits (128 vectors, 128 destinations, 32
updates per launch) are crossed in combinations no hand-written case lists."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, adagrad_slack, rel_err, rel_err_beyond, to_device, to_host

pytestmark = pytest.mark.gpu

SIZES = [1, 7, 8, 9, 255, 2048, 2049, 4099, 65536 + 5, 262143, 262144, 262151, 300011, 524288 + 8]


def _draw(case):
    rng = np.random.default_rng(1000 + case)
    lam = int(rng.choice([1, 2, 3, 4, 6, 8, 12, 16, 24, 30, 48, 54, 64, 96, 128]))
    divisors = [d for d in range(1, lam + 1) if lam // d >= 1 and lam // d <= 128]
    n = int(rng.choice(divisors))
    c = lam // n
    mode = int(rng.choice([synth.SOFTSYNC_ROUNDS, synth.SOFTSYNC_TIMED] + ([synth.HARDSYNC] if n == 1 else [])))
    fanins = [0] + [k for k in range(1, c + 1) if c % k == 0 and lam % k == 0]
    fanin = int(rng.choice(fanins))
    return dict(
        lam=lam, n=n, c=c, mode=mode, fanin=fanin, N=int(rng.choice(SIZES)),
        policy=int(rng.integers(0, 3)), opt=int(rng.integers(0, 2)), dtype=int(rng.integers(0, 2)),
        momentum=float(rng.choice([0.0, 0.9])), wd=float(rng.choice([0.0, 5e-4])),
        downcast=bool(rng.integers(0, 2)) and mode != synth.HARDSYNC, copy=bool(rng.integers(0, 2)),
        max_window=int(rng.choice([0, 0, 1, 3, 7])), seed=int(rng.integers(1, 2**31)),
        spread=float(rng.choice([0.0, 0.3, 1.0])),
    )


@pytest.mark.parametrize("case", range(128))
def test_random_configuration_against_the_oracle(case):
    import torch
    from paper_1509_04210_b200 import binding as rb

    cfg = _draw(case)
    lam, n, N, k = cfg["lam"], cfg["n"], cfg["N"], cfg["fanin"]
    m = cfg["momentum"] if cfg["opt"] == ora.OPT_MOMENTUM_SGD else 0.0
    a0 = 0.02
    th0 = synth.initial_weights(N, 0.01, cfg["seed"])
    gpu = rb.ParameterServer(N, lam, n, a0, m, cfg["wd"])
    cpu = ora.OraclePS(N, lam, n, a0, m, cfg["wd"])
    gpu.set_option(rb.OPT_GRAD_DTYPE, cfg["dtype"]), cpu.set_grad_dtype(cfg["dtype"])
    gpu.set_option(rb.OPT_LR_POLICY, cfg["policy"]), cpu.set_policy(cfg["policy"])
    gpu.set_option(rb.OPT_OPTIMIZER, cfg["opt"]), cpu.set_optimizer(cfg["opt"], 1e-8)
    if cfg["copy"]:
        gpu.set_option(rb.OPT_PUSH_MODE, rb.PUSH_COPY)
    if k:
        gpu.set_option(rb.OPT_TREE_FANIN, k)
    gpu.set_weights(to_device(th0)), cpu.set_weights(th0)
    grads_np = [synth.gradient(N, l, 0, 1e-2, cfg["dtype"], cfg["seed"]) for l in range(lam)]
    grads = [to_device(g) for g in grads_np]
    slots = [torch.full((N,), -3.0, device="cuda") for _ in range(lam)]
    nevents = 60 * max(cfg["c"], 4)
    ev = rb.Scheduler(lam, n, cfg["mode"], cfg["seed"], cfg["spread"], cfg["downcast"], k).next(nevents)
    eo = ora.OracleScheduler(lam, n, cfg["mode"], cfg["seed"], cfg["spread"], cfg["downcast"], k).run(nevents)
    assert ev.tobytes() == eo.tobytes(), cfg
    rng = np.random.default_rng(cfg["seed"])
    pos, updates = 0, 0
    at_leaf, slot_want = {}, {}
    slack = np.zeros(N)
    while pos < nevents:
        batch = ev[pos:pos + int(rng.integers(1, 4 * lam + 8))]
        pos += len(batch)
        updates += gpu.run_events(batch, grads, slots, cfg["max_window"])
        for e in batch:
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == ora.PUSH:
                if k:
                    at_leaf.setdefault(l // k, []).append((grads_np[l], int(e["pulled_ts"])))
                else:
                    assert cpu.push(grads_np[l], int(e["pulled_ts"])) > 0
            elif kind == ora.RELAY:
                msg = at_leaf.pop(l)
                assert cpu.push_relay([g for g, _ in msg], [p for _, p in msg]) > 0
            elif kind == ora.STEP:
                assert cpu.step() == 1
                if cfg["opt"] == ora.OPT_ADAGRAD:
                    slack += adagrad_slack(cpu.state(), cpu.last_clock()["abar"], cfg["c"], 0.06)
            elif kind == ora.PULL:
                slot_want[l] = (cpu.pull()[0], slack.copy())
            elif kind == ora.BROADCAST:
                cur = (cpu.pull()[0], slack.copy())
                slot_want = {j: cur for j in range(lam)}
        assert gpu.timestamp() == cpu.timestamp() == updates, cfg
        if updates:
            g, o = gpu.last_clock(), cpu.last_clock()
            np.testing.assert_array_equal(g["sigma"], o["sigma"])
            np.testing.assert_array_equal(g["pulled_ts"], o["pulled_ts"])
            np.testing.assert_array_equal(g["scale"].view(np.uint32), o["scale"].view(np.uint32))
            assert g["avg_sigma"] == o["avg_sigma"]
    assert updates >= 5, cfg
    th, st = torch.empty(N, device="cuda"), torch.empty(N, device="cuda")
    gpu.export_state(th, st)
    gpu.sync()
    assert rel_err_beyond(to_host(th), cpu.pull()[0], slack) <= REL_100_STEPS, cfg
    if m or cfg["opt"] == ora.OPT_ADAGRAD:
        assert rel_err(to_host(st), cpu.state()) <= REL_100_STEPS, cfg
    for l, (want, allow) in slot_want.items():
        assert rel_err_beyond(to_host(slots[l]), want, allow) <= REL_100_STEPS, (cfg, l)
    hist = gpu.staleness_histogram()
    assert int(hist.sum()) == updates * cfg["c"]
    gpu.close()
