"""Pins for the oracle's learner-event model: the staleness sets the paper prints (Section 5.1),
the timestamp rules of Section 3.1, a from-scratch replay in Python, and the generator's
published test vectors."""
import math
import os

import numpy as np
import pytest

from oracle import rudra_oracle as ora

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def _pushes(ev):
    return ev[ev["kind"] == ora.PUSH]


def test_splitmix64_published_vectors():
    for row in _rows("splitmix64_vectors.txt"):
        seed, want = int(row[0]), [int(x) for x in row[1:]]
        assert [int(x) for x in ora.splitmix64(seed, len(want))] == want


@pytest.mark.parametrize("row", _rows("staleness_section_5_1.txt"))
def test_staleness_sets_printed_in_section_5_1(row):
    # The paper measured these on a homogeneous cluster.  Two learner models bracket that: fixed
    # rounds with a seeded push order, and timed learners with a small spread of compute times.
    # Each must stay inside the printed set with the printed mean; together they produce all of it.
    lam, n, smin, smax, mean_target, mean_tol = int(row[0]), int(row[1]), int(row[2]), int(row[3]), float(row[4]), float(row[5])
    seen = set()
    for mode, spread in ((ora.SOFTSYNC_ROUNDS, 0.0), (ora.SOFTSYNC_TIMED, 0.1)):
        ev = ora.OracleScheduler(lam, n, mode, seed=7, lognormal_sigma=spread).run(150000)
        p = _pushes(ev)
        sigma = (p["ts"] - p["pulled_ts"]).astype(np.int64)
        steady = sigma[2 * lam:]                 # the first pushes all start from timestamp 0
        assert steady.min() >= smin
        assert (steady > smax).mean() < 1e-4     # "only with a very low probability (< 0.0001)"
        if n <= 2:
            assert steady.max() <= smax
        assert abs(steady.mean() - mean_target) <= mean_tol
        seen |= set(int(x) for x in np.unique(steady))
    if n <= 2:
        assert seen == set(range(smin, smax + 1))   # every printed value occurs


def test_hardsync_staleness_is_always_zero_and_weights_are_broadcast():
    lam = 7
    ev = ora.OracleScheduler(lam, 1, ora.HARDSYNC, seed=1).run(900)
    p = _pushes(ev)
    assert np.all(p["ts"] == p["pulled_ts"])
    kinds = list(ev["kind"])
    for i, k in enumerate(kinds[:-1]):
        if k == ora.STEP:
            assert kinds[i + 1] == ora.BROADCAST
    assert ora.PULL not in kinds and ora.PULL_SKIP not in kinds
    steps = ev[ev["kind"] == ora.STEP]
    assert list(steps["ts"]) == list(range(1, len(steps) + 1))
    assert len(p) // lam - len(steps) in (0, 1)


def test_single_learner_degenerates_to_zero_staleness():
    # with lambda = 1 the n-softsync protocol is hardsync (Section 5.2)
    ev = ora.OracleScheduler(1, 1, ora.SOFTSYNC_ROUNDS, seed=5).run(300)
    p = _pushes(ev)
    assert np.all(p["ts"] == p["pulled_ts"])
    assert (ev["kind"] == ora.PULL).sum() == (ev["kind"] == ora.STEP).sum()


@pytest.mark.parametrize("lam,n", [(4, 1), (4, 2), (4, 4), (30, 4), (54, 18), (60, 4), (128, 4), (5, 3), (9, 2)])
def test_rounds_invariants_and_staleness_bound(lam, n):
    c = lam // n
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_ROUNDS, seed=11).run(40 * lam * 3)
    p = _pushes(ev)
    P = np.arange(1, len(p) + 1)
    # timestamp = floor(pushes handled / c); a push sees the timestamp before its own update
    np.testing.assert_array_equal(p["ts"], (P - 1) // c)
    assert np.all(p["pulled_ts"] <= p["ts"])
    steps = ev[ev["kind"] == ora.STEP]
    np.testing.assert_array_equal(steps["ts"], np.arange(1, len(steps) + 1))   # +1 per update
    assert len(p) // c - len(steps) in (0, 1)   # the trace may end between a push and its update
    # every learner pushes exactly once per round
    full = (len(p) // lam) * lam
    rounds = p["learner"][:full].reshape(-1, lam)
    assert np.all(np.sort(rounds, axis=1) == np.arange(lam))
    # mini-batch counters
    for l in range(lam):
        np.testing.assert_array_equal(p["seq"][p["learner"] == l], np.arange((p["learner"] == l).sum()))
    sigma = (p["ts"] - p["pulled_ts"]).astype(np.int64)
    # between a learner's pull and its next push lie at most 2*lambda - 2 other pushes
    assert sigma.max() <= math.ceil((2 * lam - 2) / c)
    if lam % n == 0:
        assert sigma.max() <= 2 * n           # the paper's 2n bound (Section 3.1)
    assert abs(sigma[2 * lam:].mean() - (lam - 1) / c) <= 0.5


def test_rounds_replay_from_scratch():
    # Take only the push order from the trace and recompute everything else with a tiny model
    # written here: server timestamp, each learner's local timestamp, pull vs inquiry skip.
    lam, n = 6, 2
    c = lam // n
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_ROUNDS, seed=99).run(2000)
    order = [int(e["learner"]) for e in ev if e["kind"] == ora.PUSH]
    ts, local, count, expect = 0, [0] * lam, 0, []
    for l in order:
        expect.append((ora.PUSH, l, local[l], ts))
        count += 1
        if count % c == 0:
            ts += 1
            expect.append((ora.STEP, l, 0, ts))
        if local[l] == ts:
            expect.append((ora.PULL_SKIP, l, 0, ts))
        else:
            local[l] = ts
            expect.append((ora.PULL, l, 0, ts))
    got = [(int(e["kind"]), int(e["learner"]), int(e["pulled_ts"]), int(e["ts"])) for e in ev]
    assert got == expect[: len(got)]
    assert any(k == ora.PULL_SKIP for k, *_ in got) and any(k == ora.PULL for k, *_ in got)


def test_downcast_refreshes_every_copy_and_keeps_the_integers():
    lam, n = 8, 2
    a = ora.OracleScheduler(lam, n, ora.SOFTSYNC_ROUNDS, seed=4).run(3000)
    b = ora.OracleScheduler(lam, n, ora.SOFTSYNC_ROUNDS, seed=4, downcast=True).run(3000)
    pa, pb = _pushes(a), _pushes(b)
    m = min(len(pa), len(pb))
    # a learner's gradient timestamp is the server's when it starts its mini-batch, either way
    for f in ("learner", "pulled_ts", "ts", "seq"):
        np.testing.assert_array_equal(pa[f][:m], pb[f][:m])
    assert (b["kind"] == ora.PULL).sum() == 0
    assert (b["kind"] == ora.BROADCAST).sum() == (b["kind"] == ora.STEP).sum()


def test_permutations_are_uniform_enough():
    lam = 4
    ev = ora.OracleScheduler(lam, 1, ora.SOFTSYNC_ROUNDS, seed=2).run(24 * 400 * 10)
    p = _pushes(ev)
    full = (len(p) // lam) * lam
    rounds = [tuple(r) for r in p["learner"][:full].reshape(-1, lam)]
    counts = {}
    for r in rounds:
        counts[r] = counts.get(r, 0) + 1
    assert len(counts) == 24
    exp = len(rounds) / 24.0
    chi2 = sum((v - exp) ** 2 / exp for v in counts.values())
    assert chi2 < 60.0                         # 23 degrees of freedom; 60 is far in the tail


def test_seeds_are_deterministic_and_distinct():
    a = ora.OracleScheduler(9, 3, ora.SOFTSYNC_ROUNDS, seed=123).run(500)
    b = ora.OracleScheduler(9, 3, ora.SOFTSYNC_ROUNDS, seed=123).run(500)
    c = ora.OracleScheduler(9, 3, ora.SOFTSYNC_ROUNDS, seed=124).run(500)
    assert a.tobytes() == b.tobytes()
    assert a.tobytes() != c.tobytes()


def test_timed_mode_order_clock_and_lognormal_times():
    lam, n, s = 60, 4, 0.3
    c = lam // n
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_TIMED, seed=31, lognormal_sigma=s).run(200000)
    p = _pushes(ev)
    t = p["tick"].astype(np.int64)
    assert np.all(np.diff(t) >= 0)                                   # handled in time order
    same = np.diff(t) == 0
    assert np.all(np.diff(p["learner"].astype(np.int64))[same] > 0)  # ties by learner id
    P = np.arange(1, len(p) + 1)
    np.testing.assert_array_equal(p["ts"], (P - 1) // c)
    assert np.all(p["pulled_ts"] <= p["ts"])
    # compute times: ln(D / 2^20) ~ N(0, s)
    d = []
    for l in range(lam):
        tl = t[p["learner"] == l]
        d.append(np.diff(np.concatenate([[0], tl])))
    logd = np.log(np.concatenate(d) / 2.0 ** 20)
    assert abs(logd.mean()) < 0.01 and abs(logd.std() - s) < 0.01
    sigma = (p["ts"] - p["pulled_ts"]).astype(np.int64)[2 * lam:]
    assert abs(sigma.mean() - n) <= 1.0                              # <sigma> = n (Section 5.1)
    # with learners of roughly equal speed, sigma passes 2n only with tiny probability (Section 5.1)
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_TIMED, seed=31, lognormal_sigma=0.1).run(200000)
    p = _pushes(ev)
    sigma = (p["ts"] - p["pulled_ts"]).astype(np.int64)[2 * lam:]
    assert (sigma > 2 * n).mean() < 1e-4


def test_timed_mode_homogeneous_limit_matches_rounds_bound():
    # zero spread: all learners take equal time, ties resolve by id -> behaves like fixed rounds
    lam, n = 12, 3
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_TIMED, seed=1, lognormal_sigma=0.0).run(3000)
    p = _pushes(ev)
    full = (len(p) // lam) * lam
    np.testing.assert_array_equal(p["learner"][:full].reshape(-1, lam), np.tile(np.arange(lam), (full // lam, 1)))
    sigma = (p["ts"] - p["pulled_ts"]).astype(np.int64)
    assert sigma.max() <= 2 * n


def test_invalid_arguments():
    with pytest.raises(ValueError):
        ora.OracleScheduler(4, 5)
    with pytest.raises(ValueError):
        ora.OracleScheduler(4, 2, ora.HARDSYNC)
    with pytest.raises(ValueError):
        ora.OraclePS(0, 4, 1, 0.1, 0.0, 0.0)
