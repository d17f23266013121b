"""Pins of the oracle's update rule against library routines: where the reading of the paper's
"momentum" and "weight regularization penalty" (Section 4.2) and of AdaGrad (Section 5.5) reduces to
a textbook optimizer, the oracle must walk the same trajectory as ``torch.optim.SGD`` /
``torch.optim.Adagrad`` run in float64 on the mean gradient of each group.  Nothing here is
computed by the oracle itself, and the optimizers are torch's, not restated.

Special case used: the paper's own rate policy (Eq. 6, one rate alpha0/n for every gradient), so
the group's rate is a constant and Eq. 5's sum is the rate times the plain mean of the c gradients.
With the rate inside the velocity, v_oracle = rate * buf_torch at every step.
"""
import numpy as np
import pytest
import torch

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

F32 = lambda x: float(np.float32(x))  # noqa: E731  (the oracle takes its scalars as fp32)


def _run_oracle(N, lam, n, a0, m, wd, K, opt, grads):
    ps = ora.OraclePS(N, lam, n, a0, m, wd)
    if opt == "adagrad":
        ps.set_optimizer(ora.OPT_ADAGRAD, 1e-8)
    th0 = synth.initial_weights(N, 0.01, 11)
    ps.set_weights(th0)
    traj = []
    for k in range(K):
        for g in grads[k]:
            ps.push(g, ps.timestamp())
        assert ps.step() == 1
        traj.append((ps.pull()[0].astype(np.float64), ps.state().astype(np.float64)))
    return th0.astype(np.float64), traj


def _grads(N, c, K, std=1e-2):
    return [[synth.gradient(N, l, k, std) for l in range(c)] for k in range(K)]


@pytest.mark.parametrize("m,wd", [(0.9, 0.1), (0.5, 0.0), (0.0, 0.2), (0.0, 0.0)])
def test_momentum_weight_decay_trajectory_is_torch_sgd(m, wd):
    N, lam, n, a0, K = 96, 6, 2, 0.1, 25
    c = lam // n
    grads = _grads(N, c, K)
    th0, traj = _run_oracle(N, lam, n, a0, m, wd, K, "sgd", grads)
    rate = F32(a0) / n
    p = torch.nn.Parameter(torch.tensor(th0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=rate, momentum=F32(m), weight_decay=F32(wd), dampening=0.0, nesterov=False)
    for k in range(K):
        p.grad = torch.tensor(np.mean(np.stack(grads[k]).astype(np.float64), axis=0))
        opt.step()
        want = p.detach().numpy()
        got, vel = traj[k]
        # fp32 storage of weights and velocity after every update: a few roundings per step,
        # carried forward by the momentum's geometric sum
        tol = 8 * (k + 1) * np.finfo(np.float32).eps * np.maximum(np.abs(want), 1e-2) / (1.0 - F32(m))
        assert np.all(np.abs(got - want) <= tol), (k, np.abs(got - want).max(), tol.min())
        if m != 0.0:
            buf = opt.state[p]["momentum_buffer"].numpy()
            assert np.all(np.abs(vel - rate * buf) <= tol), (k, np.abs(vel - rate * buf).max())
    # the pin has teeth: without the penalty, or with it scaled by the rate twice, the end point differs visibly
    if wd != 0.0:
        assert np.abs(traj[-1][0] - th0).max() > 1e-3


@pytest.mark.parametrize("wd", [0.0, 0.05])
def test_adagrad_trajectory_is_torch_adagrad(wd):
    N, lam, n, a0, K = 96, 6, 2, 0.1, 25
    c = lam // n
    grads = _grads(N, c, K)
    th0, traj = _run_oracle(N, lam, n, a0, 0.0, wd, K, "adagrad", grads)
    rate = F32(a0) / n
    p = torch.nn.Parameter(torch.tensor(th0, dtype=torch.float64))
    opt = torch.optim.Adagrad([p], lr=rate, lr_decay=0.0, weight_decay=F32(wd), initial_accumulator_value=0.0,
                              eps=F32(1e-8))
    for k in range(K):
        p.grad = torch.tensor(np.mean(np.stack(grads[k]).astype(np.float64), axis=0))
        opt.step()
        want = p.detach().numpy()
        got, h = traj[k]
        # every step moves a weight by about the rate; the fp32 rounding of the c weights s_l / abar
        # and of the stored sum of squares shifts a step by a few parts in 1e7
        tol = 16 * (k + 1) * np.finfo(np.float32).eps * np.maximum(np.abs(want), rate)
        assert np.all(np.abs(got - want) <= tol), (k, np.abs(got - want).max(), tol.min())
        hs = opt.state[p]["sum"].numpy()
        assert np.all(np.abs(h - hs) <= 16 * (k + 1) * np.finfo(np.float32).eps * np.maximum(hs, 1e-12)), k


def test_library_pins_separate_the_alternative_readings():
    """The trajectories torch gives for the rejected readings (penalty scaled by the rate a second
    time; penalty left out) are far outside the tolerance used above, so the pins above would
    fail an oracle that took one of them."""
    N, lam, n, a0, m, wd, K = 96, 6, 2, 0.1, 0.9, 0.1, 25
    grads = _grads(N, lam // n, K)
    th0, traj = _run_oracle(N, lam, n, a0, m, wd, K, "sgd", grads)
    rate = F32(a0) / n
    for alt_wd in (0.0, rate * F32(wd)):
        p = torch.nn.Parameter(torch.tensor(th0, dtype=torch.float64))
        opt = torch.optim.SGD([p], lr=rate, momentum=F32(m), weight_decay=alt_wd)
        for k in range(K):
            p.grad = torch.tensor(np.mean(np.stack(grads[k]).astype(np.float64), axis=0))
            opt.step()
        gap = np.abs(p.detach().numpy() - traj[-1][0]).max()
        assert gap > 1e-4, gap
