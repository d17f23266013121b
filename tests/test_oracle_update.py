"""Pins for the oracle's update rule: closed forms, invariants and special cases fixed by the
paper's equations (Eq. 2-6) and by mathematics, none of them computed by the oracle itself."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

F32_EPS = float(np.finfo(np.float32).eps)


def _mk(N, lam, n, a0, m=0.0, wd=0.0, seed=3):
    ps = ora.OraclePS(N, lam, n, a0, m, wd)
    th0 = synth.initial_weights(N, 0.01, seed)
    ps.set_weights(th0)
    return ps, th0.astype(np.float64)


def _close(got, want, scale, ulps=4.0):
    """|got - want| within a few fp32 roundings of the magnitudes involved."""
    tol = ulps * F32_EPS * np.maximum(np.abs(want), scale)
    bad = np.abs(got.astype(np.float64) - want) > tol
    assert not bad.any(), (np.abs(got - want).max(), tol.min())


def test_eq3_hardsync_is_plain_averaged_minibatch_sgd():
    # Eq. 3: theta' = theta - alpha * (1/lambda) * sum_l grad_l ; n = 1, no momentum, no decay
    N, lam, a0 = 257, 4, 0.01
    ps, th0 = _mk(N, lam, 1, a0)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(lam)]
    for g in gs:
        ps.push(g, 0)
    assert ps.step() == 1
    want = th0 - float(np.float32(a0)) * np.mean(np.stack(gs).astype(np.float64), axis=0)
    got, ts = ps.pull()
    assert ts == 1
    _close(got, want, 1e-4)
    # and it moved: a dropped gradient term or sign flip cannot pass
    assert np.abs(got - th0).max() > 1e-5
    assert np.abs((th0 + (th0 - want)) - got).max() > 1e-5


def test_eq4_eq6_lambda_softsync_is_single_gradient_step_with_alpha0_over_lambda():
    # n = lambda => c = 1: the Async rule (Eq. 4) with alpha = alpha0 / n (Eq. 6)
    N, lam, a0 = 100, 30, 0.3
    ps, th0 = _mk(N, lam, lam, a0)
    g = synth.gradient(N, 0, 0, 1e-2)
    ps.push(g, 0)
    assert ps.step() == 1
    want = th0 - (float(np.float32(a0)) / lam) * g.astype(np.float64)
    _close(ps.pull()[0], want, 1e-4)


def test_eq5_eq6_general_group_n_differs_from_c():
    # lambda = 12, n = 3 -> c = 4; step = (alpha0 / n) * mean of the 4 gradients.  n != c exposes a swap.
    N, lam, n, a0 = 64, 12, 3, 0.06
    ps, th0 = _mk(N, lam, n, a0)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(4)]
    for g in gs:
        ps.push(g, 0)
    assert ps.step() == 1
    want = th0 - (float(np.float32(a0)) / 3.0) * np.mean(np.stack(gs).astype(np.float64), axis=0)
    _close(ps.pull()[0], want, 1e-4)
    rec = ps.last_clock()
    np.testing.assert_allclose(rec["scale"], np.float32(float(np.float32(a0)) / 12.0), rtol=1e-7)
    assert abs(rec["abar"] - float(np.float32(a0)) / 3.0) < 1e-8


def test_floor_when_n_does_not_divide_lambda():
    # the paper itself runs n = 4 with lambda = 30: c = floor(30/4) = 7 (Section 5.1, Fig. 4)
    ps, _ = _mk(8, 30, 4, 0.01)
    assert ps.c == 7
    g = synth.gradient(8, 0, 0)
    for i in range(6):
        ps.push(g, 0)
        assert ps.step() == 0
    ps.push(g, 0)
    assert ps.step() == 1 and ps.timestamp() == 1


def test_identical_gradients_give_analytic_scaled_step():
    # every push carries the same g: theta_K = theta_0 - K * (alpha0/n) * g
    N, lam, n, a0, K = 33, 6, 2, 0.02, 25
    ps, th0 = _mk(N, lam, n, a0)
    g = synth.gradient(N, 0, 0, 1e-2)
    for k in range(K):
        for _ in range(3):
            ps.push(g, ps.timestamp())
        assert ps.step() == 1
    want = th0 - K * (float(np.float32(a0)) / n) * g.astype(np.float64)
    _close(ps.pull()[0], want, 1e-3, ulps=2.0 * K)
    assert ps.timestamp() == K


def test_momentum_geometric_closed_form():
    # constant g, constant rate a: v_j = a g (1 - m^j)/(1 - m); theta_K = theta_0 - sum_j v_j
    N, lam, a0, m, K = 20, 5, 0.05, 0.9, 40
    ps, th0 = _mk(N, lam, 5, a0, m=m)
    g = synth.gradient(N, 0, 0, 1e-2)
    for k in range(K):
        ps.push(g, ps.timestamp())
        ps.step()
    a = float(np.float32(a0)) / 5.0
    mm = float(np.float32(m))
    geo = sum((1.0 - mm ** j) / (1.0 - mm) for j in range(1, K + 1))
    want = th0 - a * geo * g.astype(np.float64)
    _close(ps.pull()[0], want, 1e-2, ulps=2.0 * K)
    v_want = a * g.astype(np.float64) * (1.0 - mm ** K) / (1.0 - mm)
    _close(ps.state(), v_want, 1e-4, ulps=2.0 * K)


def test_weight_decay_closed_form():
    # zero gradients, no momentum: theta_K = theta_0 * (1 - a * wd)^K with a = alpha0 / n
    N, lam, n, a0, wd, K = 50, 4, 2, 0.5, 0.25, 30
    ps, th0 = _mk(N, lam, n, a0, wd=wd)
    z = np.zeros(N, dtype=np.float32)
    for k in range(K):
        ps.push(z, ps.timestamp())
        ps.push(z, ps.timestamp())
        ps.step()
    a = float(np.float32(a0)) / n
    want = th0 * (1.0 - a * float(np.float32(wd))) ** K
    _close(ps.pull()[0], want, 0.0, ulps=2.0 * K)
    assert (1.0 - a * wd) ** K < 0.2  # the decay is large enough that dropping it would be seen


def test_momentum_and_decay_as_exact_affine_recurrence():
    # Brute force in exact rationals on a tiny vector: the state (theta, v) follows the affine map
    #   v' = m v + (u + a wd theta),  theta' = theta - v'
    # written here as a 2x2 matrix acting on (theta, v) plus a forcing term, multiplied out over K
    # steps without ever forming the per-step recurrence the oracle uses.
    N, lam, n, K = 6, 4, 2, 9
    a0, m, wd = np.float32(0.04), np.float32(0.75), np.float32(0.125)
    ps, th0 = _mk(N, lam, n, float(a0), m=float(m), wd=float(wd))
    grads = [[synth.gradient(N, l, k, 1e-2) for l in range(2)] for k in range(K)]
    for k in range(K):
        for g in grads[k]:
            ps.push(g, ps.timestamp())
        ps.step()
    s = Fraction(float(np.float32(float(a0) / 4.0)))          # per-gradient step size, fp32 as stored
    a = Fraction(float(np.float32(2 * float(np.float32(float(a0) / 4.0)))))
    mF, wF = Fraction(float(m)), Fraction(float(wd))
    A = [[1 - a * wF, -mF], [a * wF, mF]]
    got, _ = ps.pull()
    vel = ps.state()
    for k_el in range(N):
        # accumulate sum_j A^(K-1-j) * b_j + A^K x0 by Horner
        x = [Fraction(float(th0[k_el])), Fraction(0)]
        for k in range(K):
            u = sum(s * Fraction(float(g[k_el])) for g in grads[k])
            x = [A[0][0] * x[0] + A[0][1] * x[1] - u, A[1][0] * x[0] + A[1][1] * x[1] + u]
        assert abs(float(x[0]) - float(got[k_el])) <= 2 * K * F32_EPS * max(abs(float(x[0])), 1e-3)
        assert abs(float(x[1]) - float(vel[k_el])) <= 2 * K * F32_EPS * max(abs(float(x[1])), 1e-4)


def test_eq7_group_average_is_linear_and_order_free():
    # Eq. 7's argument: a step on c gradients with equal weights equals a step on their mean,
    # and the order inside the group is immaterial.
    N, lam, a0 = 128, 8, 0.1
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(8)]
    ps1, th0 = _mk(N, lam, 1, a0)
    for g in gs:
        ps1.push(g, 0)
    ps1.step()
    ps2, _ = _mk(N, lam, 1, a0)
    for g in reversed(gs):
        ps2.push(g, 0)
    ps2.step()
    ps3, _ = _mk(N, 1, 1, a0)
    ps3.push(np.mean(np.stack(gs).astype(np.float64), axis=0).astype(np.float32), 0)
    ps3.step()
    _close(ps2.pull()[0], ps1.pull()[0].astype(np.float64), 1e-4, ulps=2)
    _close(ps3.pull()[0], ps1.pull()[0].astype(np.float64), 1e-4, ulps=3)


def _advance(ps, N, k):
    z = np.zeros(N, dtype=np.float32)
    for _ in range(k):
        for _ in range(ps.c):
            ps.push(z, ps.timestamp())
        ps.step()


def test_staleness_vector_clock_and_eq2():
    # sigma = j - i (Section 3.1); <sigma> = (i-1) - mean(i_1..i_c) (Eq. 2), both ways
    N = 4
    ps, _ = _mk(N, 6, 2, 0.01)
    _advance(ps, N, 7)                      # ts = 7
    g = synth.gradient(N, 0, 0)
    for p in (7, 3, 5):
        ps.push(g, p)
    ps.step()
    rec = ps.last_clock()
    assert rec["c"] == 3
    assert list(rec["pulled_ts"]) == [7, 3, 5]
    assert list(rec["sigma"]) == [0, 4, 2]
    assert rec["avg_sigma"] == pytest.approx(7 - (7 + 3 + 5) / 3.0, abs=1e-12)
    assert rec["avg_sigma"] == pytest.approx(np.mean([0, 4, 2]), abs=1e-12)
    assert max(rec["pulled_ts"]) < ps.timestamp()   # every clock entry precedes the new timestamp
    assert ps.timestamp() == 8


def test_future_timestamp_is_rejected_and_short_group_does_not_step():
    N = 4
    ps, th0 = _mk(N, 4, 2, 0.01)
    g = synth.gradient(N, 0, 0)
    assert ps.push(g, 1) < 0                # weights with timestamp 1 do not exist yet
    assert ps.push(g, 0) == 1
    assert ps.step() == 0 and ps.timestamp() == 0
    np.testing.assert_array_equal(ps.pull()[0], th0.astype(np.float32))


def test_fifo_exactly_c_per_update():
    # three queued with c = 2: the third belongs to the next group
    N = 16
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(4)]
    ps, th0 = _mk(N, 4, 2, 0.2)
    for g in gs[:3]:
        ps.push(g, 0)
    assert ps.step() == 1 and ps.step() == 0
    a = float(np.float32(0.2)) / 2
    want1 = th0 - a * (gs[0].astype(np.float64) + gs[1]) / 2
    _close(ps.pull()[0], want1, 1e-4)
    ps.push(gs[3], 1)
    assert ps.step() == 1
    assert list(ps.last_clock()["sigma"]) == [1, 0]
    want2 = ps_w = want1 - a * (gs[2].astype(np.float64) + gs[3]) / 2
    _close(ps.pull()[0], want2, 1e-4, ulps=6)


def test_per_gradient_policy_divides_by_each_staleness():
    # the footnote variant of Section 5.1: staler gradients get smaller rates; sigma = 0 floors at 1
    N, a0 = 8, 0.12
    ps, _ = _mk(N, 6, 2, a0)
    ps.set_policy(ora.LR_PER_GRADIENT)
    _advance(ps, N, 6)
    th = ps.pull()[0].astype(np.float64)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(3)]
    for g, p in zip(gs, (6, 2, 5)):         # sigma = 0, 4, 1
        ps.push(g, p)
    ps.step()
    a = float(np.float32(a0))
    want_scales = [a / (1 * 3), a / (4 * 3), a / (1 * 3)]
    rec = ps.last_clock()
    np.testing.assert_allclose(rec["scale"], want_scales, rtol=1e-7)
    want = th - sum(s * g.astype(np.float64) for s, g in zip(want_scales, gs))
    _close(ps.pull()[0], want, 1e-4)


def test_group_mean_policy_divides_by_measured_average_staleness():
    N, a0 = 8, 0.12
    ps, _ = _mk(N, 6, 2, a0)
    ps.set_policy(ora.LR_GROUP_MEAN)
    _advance(ps, N, 6)
    th = ps.pull()[0].astype(np.float64)
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(3)]
    for g, p in zip(gs, (6, 2, 3)):         # sigma = 0, 4, 3 -> <sigma> = 7/3
        ps.push(g, p)
    ps.step()
    a = float(np.float32(a0))
    want = th - (a / (7.0 / 3.0)) * np.mean(np.stack(gs).astype(np.float64), axis=0)
    _close(ps.pull()[0], want, 1e-4)
    # <sigma> below 1 floors at 1
    for g in gs:
        ps.push(g, ps.timestamp())
    th = ps.pull()[0].astype(np.float64)
    ps.step()
    want = th - a * np.mean(np.stack(gs).astype(np.float64), axis=0)
    _close(ps.pull()[0], want, 1e-4)


def test_bf16_gradients_widen_exactly():
    N = 300
    gs32 = [synth.gradient(N, l, 0, 1e-3) for l in range(2)]
    bits = [synth.to_bf16_bits(g) for g in gs32]
    wide = [synth.bf16_bits_to_f32(b) for b in bits]
    # the rounding recipe itself: within half a bf16 ulp, and idempotent
    for g, w in zip(gs32, wide):
        assert np.all(np.abs(w - g) <= np.abs(g) * 2.0 ** -8)
        np.testing.assert_array_equal(synth.to_bf16_bits(w), synth.to_bf16_bits(g))
    a, _ = _mk(N, 2, 1, 0.01, m=0.9, wd=5e-4)
    b, _ = _mk(N, 2, 1, 0.01, m=0.9, wd=5e-4)
    a.set_grad_dtype(ora.GRAD_BF16)
    for x, y in zip(bits, wide):
        a.push(x, 0)
        b.push(y, 0)
    a.step(), b.step()
    np.testing.assert_array_equal(a.pull()[0], b.pull()[0])


def test_adagrad_constant_gradient_closed_form():
    # constant g, no decay: h_K = K g^2 and theta_K = theta_0 - a * sum_j g / (sqrt(j) |g| + eps)
    N, K, a0 = 10, 12, 0.3
    ps, th0 = _mk(N, 3, 3, a0)
    ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    g = synth.gradient(N, 0, 0, 1e-2)
    for _ in range(K):
        ps.push(g, ps.timestamp())
        ps.step()
    a = float(np.float32(a0)) / 3
    g64 = g.astype(np.float64)
    eps = float(np.float32(1e-8))
    want = th0 - a * sum(g64 / (np.sqrt(j) * np.abs(g64) + eps) for j in range(1, K + 1))
    _close(ps.pull()[0], want, 1e-2, ulps=2.0 * K)
    _close(ps.state(), K * g64 * g64, 0.0, ulps=2.0 * K)


def _adagrad_reference(th0, grads_per_step, weights_per_step, abar_per_step, wd, eps, digits=60):
    """Reading of AdaGrad at the server carried out in 60-digit decimal arithmetic, one weight at a
    time: gbar = sum_l w_l g_l + wd theta;  h += gbar^2;  theta -= abar gbar / (sqrt(h) + eps)."""
    from decimal import Decimal, getcontext

    getcontext().prec = digits
    D = lambda x: Decimal(float(x))
    th = [D(x) for x in th0]
    h = [Decimal(0)] * len(th)
    for grads, weights, abar in zip(grads_per_step, weights_per_step, abar_per_step):
        for k in range(len(th)):
            gbar = sum((Decimal(w) * D(g[k]) for w, g in zip(weights, grads)), Decimal(0)) + D(wd) * th[k]
            h[k] = h[k] + gbar * gbar
            th[k] = th[k] - Decimal(abar) * gbar / (h[k].sqrt() + D(eps))
    return np.array([float(x) for x in th]), np.array([float(x) for x in h])


def test_adagrad_decay_only_follows_the_scalar_recurrence():
    # g = 0, wd > 0: the only force is the L2 penalty, gbar = wd theta.  The first step is then
    # theta_1 = theta_0 - abar theta_0 / (|theta_0| + eps / wd): every weight moves towards zero by (almost
    # exactly) abar whatever its size; later steps follow the scalar recurrence, evaluated in decimal.
    N, K, a0, wd = 12, 7, 0.003, 0.25
    ps, th0 = _mk(N, 4, 2, a0, wd=wd)
    ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    z = np.zeros(N, dtype=np.float32)
    abar = float(np.float32(2 * float(np.float32(float(np.float32(a0)) / 4.0))))
    ps.push(z, 0), ps.push(z, 0)
    assert ps.step() == 1
    th1 = ps.pull()[0].astype(np.float64)
    np.testing.assert_allclose(th0 - th1, abar * np.sign(th0), rtol=1e-4)      # moved by abar towards zero
    for _ in range(K - 1):
        ps.push(z, ps.timestamp()), ps.push(z, ps.timestamp())
        assert ps.step() == 1
    want_th, want_h = _adagrad_reference(th0, [[z, z]] * K, [["0.5", "0.5"]] * K, [repr(abar)] * K,
                                         np.float32(wd), np.float32(1e-8))
    _close(ps.pull()[0], want_th, 1e-3, ulps=4.0 * K)
    _close(ps.state(), want_h, 0.0, ulps=4.0 * K)
    assert np.all(want_h > 0)            # a dropped penalty term would leave h = 0 and theta unmoved


def test_adagrad_first_step_direction_is_the_sign_of_gradient_plus_decay():
    # From h = 0 the first AdaGrad step is abar gbar / (|gbar| + eps) = abar sign(gbar): its direction
    # reveals gbar's sign.  theta = 1, g = -0.05, wd = 0.1, abar = 0.1: g + wd theta = +0.05 (weight falls);
    # without the penalty, or with the penalty taken at abar wd, gbar would be negative (weight rises).
    N = 4
    a0, wd = 0.1, 0.1
    ps = ora.OraclePS(N, 1, 1, a0, 0.0, wd)
    ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    ps.set_weights(np.array([1.0, -1.0, 1.0, -1.0], dtype=np.float32))
    ps.push(np.array([-0.05, 0.05, -0.2, 0.2], dtype=np.float32), 0)
    assert ps.step() == 1
    got = ps.pull()[0].astype(np.float64)
    a = float(np.float32(a0))
    # weights 0, 1: the penalty wins (+0.05 / -0.05); weights 2, 3: the gradient wins (-0.1 / +0.1)
    np.testing.assert_allclose(got, [1.0 - a, -1.0 + a, 1.0 + a, -1.0 - a], rtol=1e-6)


def test_adagrad_per_gradient_weights_are_step_sizes_over_their_sum():
    # c = 3 under the per-gradient policy with staleness (0, 4, 1): divisors (1, 4, 1), step sizes
    # a/3, a/12, a/3, their sum abar = 3a/4, weights s_l / abar = 4/9, 1/9, 4/9.
    # Direction pin: g = (1, -3, 1) x has weighted mean +5x/9 but plain mean -x/3, so the first step
    # (abar sign(gbar)) goes opposite ways under the two weightings.
    N, a0 = 6, 0.12
    ps, _ = _mk(N, 6, 2, a0)
    ps.set_policy(ora.LR_PER_GRADIENT)
    _advance(ps, N, 6)                                   # plain SGD on zero gradients: weights unchanged, ts = 6
    ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    th = ps.pull()[0].astype(np.float64)
    x = np.float32(0.01) * np.array([1, -1, 2, -2, 3, -3], dtype=np.float32)
    gs = [x, np.float32(-3) * x, x]
    for g, p in zip(gs, (6, 2, 5)):
        ps.push(g, p)
    assert ps.step() == 1
    rec = ps.last_clock()
    assert list(rec["sigma"]) == [0, 4, 1]
    a = float(np.float32(a0))
    assert rec["abar"] == pytest.approx(0.75 * a, rel=1e-6)
    got = ps.pull()[0].astype(np.float64)
    np.testing.assert_allclose(th - got, 0.75 * a * np.sign(x), rtol=1e-5)
    # Second step on the same group (now stale by 1, 5, 2 -> divisors 1, 5, 2): sizes matter too.
    for g, p in zip(gs, (6, 2, 5)):
        ps.push(g, p)
    assert ps.step() == 1
    assert list(ps.last_clock()["sigma"]) == [1, 5, 2]
    s2 = [float(np.float32(a / (d * 3))) for d in (1, 5, 2)]
    abar2 = float(np.float32(sum(s2)))
    want_th, want_h = _adagrad_reference(
        th, [gs, gs], [["0.4444444444444444444444", "0.1111111111111111111111", "0.4444444444444444444444"],
                       [repr(s / abar2) for s in s2]],
        [repr(float(np.float32(sum(float(np.float32(a / (d * 3))) for d in (1, 4, 1))))), repr(abar2)], 0.0, np.float32(1e-8))
    _close(ps.pull()[0], want_th, 1e-3, ulps=16.0)
    _close(ps.state(), want_h, 0.0, ulps=16.0)
    assert abs(abar2 / a - (1 / 3 + 1 / 15 + 1 / 6)) < 1e-6


def test_adagrad_brute_force_on_a_tiny_vector():
    # Everything at once on 5 weights: three gradients per update with unequal staleness, weight
    # decay, changing rates; decimal arithmetic, divisors and weights worked out here from the
    # staleness the test itself imposes.
    N, a0, wd, K = 5, 0.09, 0.05, 6
    ps, _ = _mk(N, 6, 2, a0, wd=wd, seed=11)
    ps.set_policy(ora.LR_PER_GRADIENT)
    ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    th0 = ps.pull()[0].astype(np.float64)
    a = float(np.float32(a0))
    grads, weights, abars = [], [], []
    for k in range(K):
        ts = ps.timestamp()
        lags = [min(ts, d) for d in (0, k, 2)]            # staleness imposed on the three gradients
        gs = [synth.gradient(N, l, k, 1e-2, seed=11) for l in range(3)]
        for g, lag in zip(gs, lags):
            ps.push(g, ts - lag)
        assert ps.step() == 1
        s = [float(np.float32(a / (max(lag, 1) * 3))) for lag in lags]
        abar = float(np.float32(sum(s)))
        grads.append(gs), weights.append([repr(x / abar) for x in s]), abars.append(repr(abar))
        assert list(ps.last_clock()["sigma"]) == lags
    want_th, want_h = _adagrad_reference(th0, grads, weights, abars, np.float32(wd), np.float32(1e-8))
    _close(ps.pull()[0], want_th, 1e-3, ulps=4.0 * K)
    _close(ps.state(), want_h, 1e-9, ulps=4.0 * K)
    # the penalty is visible at this size: the same run without it ends elsewhere
    no_wd, _ = _adagrad_reference(th0, grads, weights, abars, 0.0, np.float32(1e-8))
    assert np.abs(no_wd - want_th).max() > 50 * F32_EPS * np.abs(want_th).max()


def test_zero_rate_leaves_the_weights_where_they_are():
    # alpha0 = 0 makes every step size 0 (Eq. 6): neither optimizer may move a weight, and nothing
    # may turn into NaN.  AdaGrad's sum of squares still grows, by the square of Eq. 5's plain mean.
    N = 9
    gs = [synth.gradient(N, l, 0, 1e-2) for l in range(3)]
    for opt in (ora.OPT_MOMENTUM_SGD, ora.OPT_ADAGRAD):
        ps, th0 = _mk(N, 3, 1, 0.0, m=0.9 if opt == ora.OPT_MOMENTUM_SGD else 0.0)
        ps.set_optimizer(opt, 1e-8)
        for g in gs:
            ps.push(g, 0)
        assert ps.step() == 1
        np.testing.assert_array_equal(ps.pull()[0], th0.astype(np.float32))
        if opt == ora.OPT_ADAGRAD:
            mean = np.mean(np.stack(gs).astype(np.float64), axis=0)
            _close(ps.state(), mean * mean, 0.0, ulps=4)
        else:
            np.testing.assert_array_equal(ps.state(), np.zeros(N, dtype=np.float32))


def test_strict_fp32_mode_tracks_the_double_mode():
    # the fp32 evaluation is the same rule: after a few updates it differs only by fp32 rounding
    N, lam, n = 500, 6, 2
    for opt in (ora.OPT_MOMENTUM_SGD, ora.OPT_ADAGRAD):
        a, _ = _mk(N, lam, n, 0.02, m=0.9 if opt == ora.OPT_MOMENTUM_SGD else 0.0, wd=5e-4)
        b, _ = _mk(N, lam, n, 0.02, m=0.9 if opt == ora.OPT_MOMENTUM_SGD else 0.0, wd=5e-4)
        for ps in (a, b):
            ps.set_optimizer(opt, 1e-8)
            ps.set_policy(ora.LR_PER_GRADIENT)
        b.set_strict(True)
        for k in range(10):
            for l in range(3):
                g = synth.gradient(N, l, k, 1e-2)
                p_ts = max(0, a.timestamp() - l)
                a.push(g, p_ts)
                b.push(g, p_ts)
            assert a.step() == 1 and b.step() == 1
        ta, tb = a.pull()[0].astype(np.float64), b.pull()[0].astype(np.float64)
        rms = np.sqrt(np.mean(ta * ta))
        assert np.max(np.abs(ta - tb) / np.maximum(np.abs(ta), rms)) < 2e-6
        assert not np.array_equal(a.pull()[0], b.pull()[0]) or opt == ora.OPT_ADAGRAD
