"""Host-side checks that need no GPU: the library loads and exports what the header declares,
its scheduler reproduces the oracle's event trace bit for bit, and argument errors are reported
before any device work."""
import os
import re

import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import binding as rb
from paper_1509_04210_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(rudra_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    L = rb.lib()
    names = _declared_symbols()
    assert len(names) >= 24
    for name in names:
        assert hasattr(L, name), name


def test_library_exports_nothing_but_its_interface():
    import subprocess

    out = subprocess.check_output(["nm", "-D", "--defined-only", rb.library_path()], text=True)
    exported = {line.split()[-1] for line in out.splitlines() if " T " in line}
    declared = set(_declared_symbols())
    extra = sorted(n for n in exported if n.startswith("rudra") and n not in declared)
    assert not extra, extra                       # e.g. the benchmark's probe lives in a library of its own


def test_header_constants_match_binding():
    text = open(os.path.join(ROOT, "include", "rudra_ps.h")).read()
    defs = {k: int(v.strip("()")) for k, v in re.findall(r"#define\s+(RUDRA_[A-Z0-9_]+)\s+(\(?-?\d+\)?)", text)}
    assert defs["RUDRA_MAX_GROUP"] == rb.MAX_GROUP and defs["RUDRA_MAX_DSTS"] == rb.MAX_DSTS
    assert defs["RUDRA_QUEUE_CAP"] == rb.QUEUE_CAP
    assert (defs["RUDRA_E_INVAL"], defs["RUDRA_E_BAD_TS"], defs["RUDRA_E_QUEUE_FULL"], defs["RUDRA_E_CUDA"],
            defs["RUDRA_E_STATE"], defs["RUDRA_E_NOMEM"]) == (rb.E_INVAL, rb.E_BAD_TS, rb.E_QUEUE_FULL, rb.E_CUDA, rb.E_STATE,
                                                             rb.E_NOMEM)
    assert defs["RUDRA_HIST_BINS"] == rb.HIST_BINS
    assert (defs["RUDRA_EV_PUSH"], defs["RUDRA_EV_STEP"], defs["RUDRA_EV_PULL"], defs["RUDRA_EV_PULL_SKIP"],
            defs["RUDRA_EV_BROADCAST"], defs["RUDRA_EV_RELAY"]) == (1, 2, 3, 4, 5, 6) == (
        ora.PUSH, ora.STEP, ora.PULL, ora.PULL_SKIP, ora.BROADCAST, ora.RELAY)
    assert (defs["RUDRA_OPT_PUSH_MODE"], defs["RUDRA_OPT_TREE_FANIN"], defs["RUDRA_PUSH_COPY"]) == (
        rb.OPT_PUSH_MODE, rb.OPT_TREE_FANIN, rb.PUSH_COPY)
    assert defs["RUDRA_GRAD_BF16"] == rb.GRAD_BF16 == synth.GRAD_BF16
    assert (defs["RUDRA_SCHED_HARDSYNC"], defs["RUDRA_SCHED_SOFTSYNC_ROUNDS"], defs["RUDRA_SCHED_SOFTSYNC_TIMED"]) == (
        synth.HARDSYNC, synth.SOFTSYNC_ROUNDS, synth.SOFTSYNC_TIMED)
    assert rb.EVENT_DTYPE.itemsize == 40 == ora.EVENT_DTYPE.itemsize


CASES = [
    (4, 1, rb.SCHED_HARDSYNC, 0.3, False),
    (4, 1, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False),
    (30, 30, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False),
    (30, 4, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False),
    (60, 4, rb.SCHED_SOFTSYNC_TIMED, 0.3, False),
    (60, 4, rb.SCHED_SOFTSYNC_TIMED, 0.0, False),
    (54, 18, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False),
    (128, 4, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, True),
    (7, 3, rb.SCHED_SOFTSYNC_TIMED, 1.0, True),
    (1, 1, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False),
    (1, 1, rb.SCHED_SOFTSYNC_TIMED, 0.3, False),
]


@pytest.mark.parametrize("lam,n,mode,spread,downcast", CASES)
@pytest.mark.parametrize("seed", [synth.MASTER_SEED, 1, 2**63 + 12345])
def test_scheduler_trace_equals_oracle_bit_for_bit(lam, n, mode, spread, downcast, seed):
    count = 20000
    a = rb.Scheduler(lam, n, mode, seed, spread, downcast).next(count)
    b = ora.OracleScheduler(lam, n, mode, seed, spread, downcast).run(count)
    assert a.tobytes() == b.tobytes()
    assert (a["kind"] == rb.EV_PUSH).sum() > count // 4


TREE_CASES = [
    (12, 2, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False, 3),
    (54, 18, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False, 3),
    (54, 3, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, False, 6),
    (128, 4, rb.SCHED_SOFTSYNC_ROUNDS, 0.3, True, 8),
    (8, 1, rb.SCHED_HARDSYNC, 0.3, False, 4),
    (60, 4, rb.SCHED_SOFTSYNC_TIMED, 0.3, False, 5),
    (6, 2, rb.SCHED_SOFTSYNC_TIMED, 0.7, True, 1),
]


@pytest.mark.parametrize("lam,n,mode,spread,downcast,fanin", TREE_CASES)
@pytest.mark.parametrize("seed", [synth.MASTER_SEED, 2**63 + 12345])
def test_tree_scheduler_trace_equals_oracle_bit_for_bit(lam, n, mode, spread, downcast, fanin, seed):
    # learners -> leaves -> root (Section 3.3): PUSH, RELAY, STEP and pull events in the same order
    count = 20000
    a = rb.Scheduler(lam, n, mode, seed, spread, downcast, fanin).next(count)
    b = ora.OracleScheduler(lam, n, mode, seed, spread, downcast, fanin).run(count)
    assert a.tobytes() == b.tobytes()
    assert (a["kind"] == rb.EV_RELAY).sum() * fanin <= (a["kind"] == rb.EV_PUSH).sum()
    assert (a["kind"] == rb.EV_RELAY).sum() > count // (8 * fanin)
    with pytest.raises(ValueError):
        rb.Scheduler(lam, n, mode, seed, spread, downcast, lam + 1)


@pytest.mark.parametrize("mode,fanin", [(rb.SCHED_SOFTSYNC_ROUNDS, 0), (rb.SCHED_SOFTSYNC_TIMED, 0), (rb.SCHED_SOFTSYNC_ROUNDS, 2)])
def test_reported_pulls_change_the_trace_the_same_way_on_both_sides(mode, fanin):
    # learner 3 loses every second pull and reports the weights it really holds: its gradients are
    # staler than the scheduler assumed.  Both schedulers must take the report the same way.
    lam, n = 12, 3
    a = rb.Scheduler(lam, n, mode, 77, 0.3, False, fanin)
    b = ora.OracleScheduler(lam, n, mode, 77, 0.3, False, fanin)
    held, lost, reported = 0, 0, 0
    stale_seen = 0
    for _ in range(6000):
        ea, eb = a.next(1)[0], b.run(1)[0]
        assert ea.tobytes() == eb.tobytes()
        if int(ea["learner"]) != 3:
            continue
        if ea["kind"] == rb.EV_PUSH:
            assert int(ea["pulled_ts"]) == held              # the push carries what the learner reported
            stale_seen = max(stale_seen, int(ea["ts"]) - held)
        elif ea["kind"] in (rb.EV_PULL, rb.EV_PULL_SKIP):
            lost += 1
            if lost % 2 == 0:
                held = int(ea["ts"])
            else:
                assert a.on_pull(3, held) == 0 and b.on_pull(3, held) == 0
                reported += 1
    assert reported > 50 and stale_seen > n
    with pytest.raises(rb.RudraError) as e:
        a.on_pull(3, 10**9)                                  # weights that do not exist yet
    assert e.value.code == rb.E_BAD_TS and b.on_pull(3, 10**9) == -2
    with pytest.raises(rb.RudraError):
        a.on_pull(lam, 0)


def test_scheduler_is_incremental():
    s1 = rb.Scheduler(9, 3, rb.SCHED_SOFTSYNC_TIMED, 5)
    whole = s1.next(999)
    s2 = rb.Scheduler(9, 3, rb.SCHED_SOFTSYNC_TIMED, 5)
    parts = np.concatenate([s2.next(k) for k in (1, 2, 500, 496)])
    assert whole.tobytes() == parts.tobytes()


def test_scheduler_rejects_bad_arguments():
    for args in [(0, 1, 1), (4, 0, 1), (4, 5, 1), (4, 2, 0), (4, 1, 7)]:
        with pytest.raises(ValueError):
            rb.Scheduler(*args)
    with pytest.raises(ValueError):
        rb.Scheduler(4, 1, rb.SCHED_SOFTSYNC_TIMED, 1, -0.5)


def test_create_rejects_bad_arguments_without_touching_the_device():
    bad = [
        (0, 4, 1, 0.1, 0.0, 0.0),
        (16, 0, 1, 0.1, 0.0, 0.0),
        (16, 4, 0, 0.1, 0.0, 0.0),
        (16, 4, 5, 0.1, 0.0, 0.0),        # n > lambda (Section 3.1: n ranges over 1..lambda)
        (16, 4, 1, -0.1, 0.0, 0.0),
        (16, 4, 1, 0.1, 1.0, 0.0),
        (16, 4, 1, 0.1, 0.5, -1.0),
        (16, 4, 1, float("nan"), 0.0, 0.0),
        (16, 1000, 1, 0.1, 0.0, 0.0),     # c = 1000 > RUDRA_MAX_GROUP
    ]
    for args in bad:
        with pytest.raises(rb.RudraError) as e:
            rb.ParameterServer(*args)
        assert e.value.code == rb.E_INVAL and len(str(e.value)) > 20


def test_null_handles_are_reported():
    L = rb.lib()
    assert L.rudra_ps_step(None) == rb.E_INVAL
    assert L.rudra_ps_push(None, None, 0) == rb.E_INVAL
    assert L.rudra_ps_timestamp(None) == rb.E_INVAL
    assert L.rudra_sched_next(None, None, 1) == rb.E_INVAL
    L.rudra_ps_destroy(None)
    L.rudra_sched_destroy(None)
    assert b"handle" in L.rudra_last_error()


def test_workload_shapes():
    w = synth.WORKLOADS
    assert w["cifar10"].nparams == 89578 and w["imagenet"].nparams == 60965224
    assert [w[k].c for k in ("tiny", "cifar10", "mid", "imagenet", "stress")] == [4, 1, 15, 3, 32]
    g = synth.gradient(1000, 3, 5, 1e-3)
    assert g.dtype == np.float32 and abs(float(g.std()) - 1e-3) < 2e-4
    np.testing.assert_array_equal(g, synth.gradient(1000, 3, 5, 1e-3))
    assert not np.array_equal(g, synth.gradient(1000, 3, 6, 1e-3))


def test_bf16_rounding_recipe_agrees_with_torch():
    # the input recipe rounds to nearest, ties to even; torch's cast is an independent implementation
    import torch

    rng = np.random.default_rng(0)
    x = (rng.standard_normal(200000) * 1e-3).astype(np.float32)
    ties = (np.arange(1, 2001, dtype=np.uint32) << np.uint32(16)) | np.uint32(0x8000)      # exactly halfway
    x = np.concatenate([x, ties.view(np.float32), -ties.view(np.float32), np.float32([0.0, -0.0, 1.0, 65504.0])])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(synth.to_bf16_bits(x), want)
    np.testing.assert_array_equal(synth.bf16_bits_to_f32(want), torch.from_numpy(x).to(torch.bfloat16).float().numpy())
