"""Pins for the oracle's two-level server tree (Section 3.3, Rudra-adv): leaves average their
learners' gradients and relay the average, the root applies the update.  The paper fixes that much;
the pins tie the rest of the reading to the flat server of Section 3.2, whose arithmetic is pinned
by Eq. 2-6, and to numbers worked out by hand."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

F32_EPS = float(np.finfo(np.float32).eps)


def _mk(N, lam, n, a0, m=0.0, wd=0.0, policy=ora.LR_PAPER_N, opt=ora.OPT_MOMENTUM_SGD, seed=3):
    ps = ora.OraclePS(N, lam, n, a0, m, wd)
    ps.set_policy(policy)
    ps.set_optimizer(opt, 1e-8)
    th0 = synth.initial_weights(N, 0.01, seed)
    ps.set_weights(th0)
    return ps, th0.astype(np.float64)


def _close(got, want, scale, ulps=4.0):
    tol = ulps * F32_EPS * np.maximum(np.abs(want), scale)
    assert not (np.abs(got.astype(np.float64) - want) > tol).any(), np.abs(got - want).max()


def _advance(ps, N, k):
    z = np.zeros(N, dtype=np.float32)
    for _ in range(k):
        for _ in range(ps.c):
            ps.push(z, ps.timestamp())
        ps.step()


@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_PER_GRADIENT, ora.LR_GROUP_MEAN])
@pytest.mark.parametrize("opt", [ora.OPT_MOMENTUM_SGD, ora.OPT_ADAGRAD])
def test_fan_in_one_is_the_flat_server_bit_for_bit(policy, opt):
    # a leaf with one learner relays that learner's gradient unchanged: nothing may differ
    N, lam, n = 37, 6, 2
    m = 0.9 if opt == ora.OPT_MOMENTUM_SGD else 0.0
    flat, _ = _mk(N, lam, n, 0.05, m, 5e-4, policy, opt)
    tree, _ = _mk(N, lam, n, 0.05, m, 5e-4, policy, opt)
    for k in range(6):
        for l in range(3):
            g = synth.gradient(N, l, k, 1e-2)
            p = max(0, flat.timestamp() - l)
            assert flat.push(g, p) == tree.push_relay([g], [p])
        assert flat.step() == 1 and tree.step() == 1
        a, b = flat.last_clock(), tree.last_clock()
        np.testing.assert_array_equal(a["scale"].view(np.uint32), b["scale"].view(np.uint32))
        np.testing.assert_array_equal(a["sigma"], b["sigma"])
        assert a["avg_sigma"] == b["avg_sigma"] and a["abar"] == b["abar"]
    np.testing.assert_array_equal(flat.pull()[0], tree.pull()[0])
    np.testing.assert_array_equal(flat.state(), tree.state())


@pytest.mark.parametrize("policy", [ora.LR_PAPER_N, ora.LR_GROUP_MEAN])
def test_equal_rates_make_the_tree_equal_the_flat_server(policy):
    # Eq. 7's argument: the mean of leaf means is the mean of all gradients when every gradient
    # gets the same rate.  c = 6 as 3 leaves of 2, against the same 6 gradients pushed directly.
    N, lam, n, K = 64, 12, 2, 8
    flat, _ = _mk(N, lam, n, 0.06, 0.9, 5e-4, policy)
    tree, _ = _mk(N, lam, n, 0.06, 0.9, 5e-4, policy)
    for k in range(K):
        ts = flat.timestamp()
        gs = [synth.gradient(N, l, k, 1e-2) for l in range(6)]
        ps_ = [max(0, ts - (l % 3)) for l in range(6)]
        for g, p in zip(gs, ps_):
            flat.push(g, p)
        for j in range(3):
            tree.push_relay(gs[2 * j: 2 * j + 2], ps_[2 * j: 2 * j + 2])
        assert flat.step() == 1 and tree.step() == 1
        a, b = flat.last_clock(), tree.last_clock()
        np.testing.assert_array_equal(a["pulled_ts"], b["pulled_ts"])      # same vector clock, same Eq. 2
        np.testing.assert_array_equal(a["sigma"], b["sigma"])
        assert a["avg_sigma"] == b["avg_sigma"]
        assert b["abar"] == pytest.approx(a["abar"], rel=2e-7)
        assert list(tree.last_messages()["fanin"]) == [2, 2, 2]
    _close(tree.pull()[0], flat.pull()[0].astype(np.float64), 1e-3, ulps=4.0 * K)
    _close(tree.state(), flat.state().astype(np.float64), 1e-4, ulps=4.0 * K)
    assert tree.timestamp() == flat.timestamp() == K


def test_relay_of_identical_gradients_is_that_gradient():
    # the average of k copies of g is g: a relay of (g, g, g, g) acts like four direct pushes of g
    N = 50
    g = synth.gradient(N, 0, 0, 1e-2)
    a, th0 = _mk(N, 4, 1, 0.1)
    b, _ = _mk(N, 4, 1, 0.1)
    for _ in range(4):
        a.push(g, 0)
    b.push_relay([g, g, g, g], [0, 0, 0, 0])
    assert a.step() == 1 and b.step() == 1
    want = th0 - float(np.float32(0.1)) * g.astype(np.float64)
    _close(a.pull()[0], want, 1e-4)
    _close(b.pull()[0], want, 1e-4)


def test_leaf_average_and_root_step_by_hand():
    # c = 4 as two leaves of two, n = 3 (lambda = 12), no momentum, no decay:
    #   theta' = theta - (alpha0 / 3) * (1/4) * (2 * mean(g0, g1) + 2 * mean(g2, g3))        (Eq. 5, Eq. 6)
    # each relayed average is multiplied by alpha0 * 2 / (3 * 4).
    N, a0 = 16, 0.12
    ps, th0 = _mk(N, 12, 3, a0)
    gs = [synth.gradient(N, l, 0, 1e-2).astype(np.float32) for l in range(4)]
    assert ps.push_relay(gs[:2], [0, 0]) == 2
    assert ps.step() == 0                                   # half a group: no update
    assert ps.push_relay(gs[2:], [0, 0]) == 4
    assert ps.step() == 1 and ps.timestamp() == 1
    a = float(np.float32(a0))
    msg = ps.last_messages()
    np.testing.assert_allclose(msg["step"], [a * 2 / 12, a * 2 / 12], rtol=1e-7)
    m01 = ((gs[0].astype(np.float64) + gs[1]) / 2).astype(np.float32).astype(np.float64)   # a 32-bit message
    m23 = ((gs[2].astype(np.float64) + gs[3]) / 2).astype(np.float32).astype(np.float64)
    want = th0 - (a / 3.0) * 0.25 * (2 * m01 + 2 * m23)
    _close(ps.pull()[0], want, 1e-4)
    assert np.abs(ps.pull()[0] - th0).max() > 1e-5


def test_per_message_rate_uses_the_mean_staleness_of_the_message():
    # per-gradient policy in the tree: one rate per relayed average, alpha0 / max(mean staleness, 1).
    # ts = 6; leaf A relays gradients pulled at (6, 2): staleness (0, 4), mean 2 -> alpha0 / 2;
    # leaf B relays (6, 5): staleness (0, 1), mean 0.5 -> floor 1 -> alpha0.  c = 4, so the
    # averages are multiplied by (alpha0 / 2) * 2/4 and alpha0 * 2/4.
    N, a0 = 8, 0.12
    ps, _ = _mk(N, 8, 2, a0, policy=ora.LR_PER_GRADIENT)
    _advance(ps, N, 6)
    th = ps.pull()[0].astype(np.float64)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(4)]
    ps.push_relay(gs[:2], [6, 2])
    ps.push_relay(gs[2:], [6, 5])
    assert ps.step() == 1
    rec, msg = ps.last_clock(), ps.last_messages()
    assert list(rec["sigma"]) == [0, 4, 0, 1] and list(rec["pulled_ts"]) == [6, 2, 6, 5]
    assert rec["avg_sigma"] == pytest.approx(6 - (6 + 2 + 6 + 5) / 4.0, abs=1e-12)        # Eq. 2 over all four
    a = float(np.float32(a0))
    np.testing.assert_allclose(msg["step"], [a / 2 * 0.5, a * 0.5], rtol=1e-7)
    np.testing.assert_allclose(rec["scale"], [a / 8, a / 8, a / 4, a / 4], rtol=1e-7)
    assert rec["abar"] == pytest.approx(0.75 * a, rel=1e-6)
    mA = ((gs[0].astype(np.float64) + gs[1]) / 2).astype(np.float32).astype(np.float64)
    mB = ((gs[2].astype(np.float64) + gs[3]) / 2).astype(np.float32).astype(np.float64)
    want = th - (a / 4) * mA - (a / 2) * mB
    _close(ps.pull()[0], want, 1e-4)


def test_relays_and_direct_pushes_share_a_group_in_arrival_order():
    # the root takes messages one at a time (Section 3.2): a learner attached to the root directly
    # and two leaves fill one group of c = 5; the vector clock lists the gradients as they arrived
    N = 12
    ps, th0 = _mk(N, 5, 1, 0.1)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(5)]
    ps.push_relay(gs[0:2], [0, 0])
    ps.push(gs[2], 0)
    assert ps.push_relay(gs[3:5], [0, 0]) == 5
    assert ps.step() == 1
    assert list(ps.last_messages()["fanin"]) == [2, 1, 2]
    a = float(np.float32(0.1))
    want = th0 - a * np.mean(np.stack(gs).astype(np.float64), axis=0)
    _close(ps.pull()[0], want, 1e-4, ulps=6)


def test_a_relay_never_straddles_two_updates_and_cannot_come_from_the_future():
    N = 4
    ps, th0 = _mk(N, 6, 2, 0.1)                              # c = 3
    g = synth.gradient(N, 0, 0)
    assert ps.push(g, 0) == 1 and ps.push(g, 0) == 2
    assert ps.push_relay([g, g], [0, 0]) < 0                 # 2 + 2 > 3: would belong to two updates
    assert ps.push_relay([g, g, g, g], [0, 0, 0, 0]) < 0     # more than a whole group
    assert ps.push_relay([g], [1]) < 0                       # weights with timestamp 1 do not exist yet
    assert ps.step() == 0
    np.testing.assert_array_equal(ps.pull()[0], th0.astype(np.float32))
    assert ps.push_relay([g], [0]) == 3 and ps.step() == 1


def test_strict_mode_tracks_the_double_mode_in_the_tree():
    N = 300
    a, _ = _mk(N, 8, 2, 0.05, 0.9, 5e-4, ora.LR_PER_GRADIENT)
    b, _ = _mk(N, 8, 2, 0.05, 0.9, 5e-4, ora.LR_PER_GRADIENT)
    b.set_strict(True)
    for k in range(8):
        ts = a.timestamp()
        for j in range(2):
            gs = [synth.gradient(N, 2 * j + i, k, 1e-2) for i in range(2)]
            p = [max(0, ts - j), max(0, ts - 2 * j)]
            a.push_relay(gs, p), b.push_relay(gs, p)
        assert a.step() == 1 and b.step() == 1
    ta, tb = a.pull()[0].astype(np.float64), b.pull()[0].astype(np.float64)
    rms = np.sqrt(np.mean(ta * ta))
    assert np.max(np.abs(ta - tb) / np.maximum(np.abs(ta), rms)) < 2e-6


# ------------------------------------------------------------------------------------------------
# scheduler: learners -> leaves -> root
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("lam,n,k,mode,spread", [(12, 2, 3, ora.SOFTSYNC_ROUNDS, 0.3), (54, 3, 6, ora.SOFTSYNC_ROUNDS, 0.3),
                                                 (8, 1, 4, ora.HARDSYNC, 0.3), (12, 3, 2, ora.SOFTSYNC_TIMED, 0.5),
                                                 (6, 2, 1, ora.SOFTSYNC_TIMED, 0.3)])
def test_tree_trace_replayed_from_scratch(lam, n, k, mode, spread):
    """Replays the trace with a few lines of Python written from the reading: learner l sends to
    leaf l // k; a leaf relays when it holds k gradients; the root updates once the relayed
    averages stand for c gradients."""
    c = lam // n
    ev = ora.OracleScheduler(lam, n, mode, 99, spread, False, fanin=k).run(4000)
    ts, at_root = 0, 0
    fill = [0] * (lam // k)
    relays = [0] * (lam // k)
    holds = [0] * lam                      # timestamp of the weights each learner computes on
    expect_relay = expect_step = None
    pushes_by_learner = [0] * lam
    for e in ev:
        kind, l = int(e["kind"]), int(e["learner"])
        if kind == ora.PUSH:
            assert expect_relay is None and expect_step is None
            assert int(e["pulled_ts"]) == holds[l] and int(e["ts"]) == ts
            assert int(e["seq"]) == pushes_by_learner[l]
            pushes_by_learner[l] += 1
            fill[l // k] += 1
            if fill[l // k] == k:
                expect_relay = l // k
        elif kind == ora.RELAY:
            assert expect_relay == l and int(e["seq"]) == relays[l] and int(e["ts"]) == ts
            relays[l] += 1
            fill[l] = 0
            expect_relay = None
            at_root += k
            if at_root % c == 0:
                expect_step = ts + 1
        elif kind == ora.STEP:
            assert expect_step == int(e["ts"])
            ts += 1
            expect_step = None
        elif kind == ora.PULL:
            assert int(e["ts"]) == ts and holds[l] != ts
            holds[l] = ts
        elif kind == ora.PULL_SKIP:
            assert int(e["ts"]) == ts and holds[l] == ts
        elif kind == ora.BROADCAST:
            assert int(e["ts"]) == ts
            holds = [ts] * lam
    assert ts == at_root // c and ts > 10
    assert sum(relays) * k == at_root


def test_tree_with_fan_in_one_is_the_flat_trace_plus_relays():
    for mode in (ora.SOFTSYNC_ROUNDS, ora.SOFTSYNC_TIMED):
        flat = ora.OracleScheduler(30, 5, mode, 7, 0.3, False).run(3000)
        tree = ora.OracleScheduler(30, 5, mode, 7, 0.3, False, fanin=1).run(6000)
        kept = tree[tree["kind"] != ora.RELAY][:3000]
        assert kept.tobytes() == flat.tobytes()
        relay = tree[tree["kind"] == ora.RELAY]
        assert len(relay) == int((tree["kind"] == ora.PUSH).sum())


def test_tree_staleness_under_rounds_is_non_negative_and_bounded():
    # gradients wait at their leaf, so staleness grows with the fan-in; in rounds mode a leaf is
    # emptied every round, so a gradient is at most one round (n updates) older than without the tree
    lam, n, k = 54, 3, 6
    c = lam // n
    ev = ora.OracleScheduler(lam, n, ora.SOFTSYNC_ROUNDS, 5, 0.3, False, fanin=k).run(20000)
    ts = 0
    waiting = {}
    worst = 0
    root = []
    for e in ev:
        kind, l = int(e["kind"]), int(e["learner"])
        if kind == ora.PUSH:
            waiting.setdefault(l // k, []).append(int(e["pulled_ts"]))
        elif kind == ora.RELAY:
            root += waiting.pop(l)
        elif kind == ora.STEP:
            assert len(root) == c
            sig = [ts - p for p in root]
            assert min(sig) >= 0
            worst = max(worst, max(sig))
            root = []
            ts += 1
    assert 0 < worst <= 3 * n


def test_tree_rejects_fan_ins_that_do_not_divide():
    with pytest.raises(ValueError):
        ora.OracleScheduler(12, 2, ora.SOFTSYNC_ROUNDS, 1, 0.3, False, fanin=4)     # c = 6 is not a multiple of 4
    with pytest.raises(ValueError):
        ora.OracleScheduler(10, 1, ora.SOFTSYNC_ROUNDS, 1, 0.3, False, fanin=4)     # 10 learners do not fill leaves of 4
