"""Seeded synthetic workloads for the parameter-server path.

This module only makes inputs (initial weights, gradient streams, workload descriptions); it
holds none of the update rule, staleness or scheduling arithmetic and loads no native library.
The gradient streams stand in for what learners training the paper's two networks would push
(Section 4.2: a ~90 K-parameter CIFAR10 network and an ImageNet network of 5 convolutional and
3 fully connected layers); the server sees only flat vectors, so only the vector length, the
learner count and the protocol parameters matter.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

MASTER_SEED = 20150914

# scheduler modes and gradient types, by their integer values in the C interface
HARDSYNC, SOFTSYNC_ROUNDS, SOFTSYNC_TIMED = 0, 1, 2
GRAD_F32, GRAD_BF16 = 0, 1


def cifar10_layer_sizes():
    """3 convolutions of 5x5 kernels (32, 32, 64 maps) on 32x32x3 input, pooled to 4x4, plus a 10-way layer."""
    convs = [(5 * 5 * 3 * 32, 32), (5 * 5 * 32 * 32, 32), (5 * 5 * 32 * 64, 64)]
    fc = [(64 * 4 * 4 * 10, 10)]
    return [w + b for w, b in convs + fc]


def imagenet_layer_sizes():
    """5 convolutions + 3 fully connected layers (two-tower grouping in conv 2, 4, 5), weights + biases."""
    convs = [(11 * 11 * 3 * 96, 96), (5 * 5 * 48 * 256, 256), (3 * 3 * 256 * 384, 384),
             (3 * 3 * 192 * 384, 384), (3 * 3 * 192 * 256, 256)]
    fcs = [(6 * 6 * 256 * 4096, 4096), (4096 * 4096, 4096), (4096 * 1000, 1000)]
    return [w + b for w, b in convs + fcs]


@dataclass(frozen=True)
class Workload:
    name: str
    nparams: int
    lam: int          # number of learners
    n: int            # splitting parameter of n-softsync
    alpha0: float
    momentum: float
    weight_decay: float
    mode: int
    updates: int
    theta_std: float
    grad_std: float
    grad_dtype: int = GRAD_F32
    downcast: bool = False      # all learner copies refreshed after every update
    lognormal_sigma: float = 0.3

    @property
    def c(self):
        return self.lam // self.n


WORKLOADS = {
    "tiny": Workload("tiny", 4096, 4, 1, 0.01, 0.0, 0.0, HARDSYNC, 100, 0.01, 1e-2),
    "cifar10": Workload("cifar10", sum(cifar10_layer_sizes()), 30, 30, 0.001, 0.9, 4e-3, SOFTSYNC_ROUNDS, 10000, 0.01, 1e-3),
    "mid": Workload("mid", 1_000_000, 60, 4, 0.01, 0.9, 5e-4, SOFTSYNC_TIMED, 2000, 0.01, 1e-3),
    "imagenet": Workload("imagenet", sum(imagenet_layer_sizes()), 54, 18, 0.01, 0.9, 5e-4, SOFTSYNC_ROUNDS, 200, 0.01, 1e-3),
    # the size Section 4.2 states for the paper's own ImageNet network (289 MB of 32-bit floats)
    "imagenet72m": Workload("imagenet72m", 72_250_000, 54, 18, 0.01, 0.9, 5e-4, SOFTSYNC_ROUNDS, 200, 0.01, 1e-3),
    "stress": Workload("stress", sum(imagenet_layer_sizes()), 128, 4, 0.01, 0.9, 5e-4, SOFTSYNC_ROUNDS, 100, 0.01, 1e-3,
                       grad_dtype=GRAD_BF16, downcast=True),
}


def _rng(seed, purpose, a=0, b=0):
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), int(purpose), int(a), int(b)])))


def to_bf16_bits(x):
    """Round fp32 values to bfloat16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def initial_weights(nparams, std=0.01, seed=MASTER_SEED):
    return _rng(seed, 1).standard_normal(nparams, dtype=np.float32) * np.float32(std)


def gradient(nparams, learner, seq, std=1e-3, dtype=GRAD_F32, seed=MASTER_SEED):
    """The gradient learner ``learner`` pushes for its mini-batch number ``seq``."""
    g = _rng(seed, 2, learner, seq).standard_normal(nparams, dtype=np.float32) * np.float32(std)
    return to_bf16_bits(g) if dtype == GRAD_BF16 else g


def device_gradient(nparams, learner, std=1e-3, dtype=GRAD_F32, seed=MASTER_SEED, device="cuda"):
    """Full-size gradient buffer generated on the device (one per learner, reused across its pushes)."""
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed((int(seed) * 1000003 + 7919 * (int(learner) + 1)) % (2**63 - 1))
    g = torch.empty(nparams, dtype=torch.float32, device=device)
    g.normal_(0.0, float(std), generator=gen)
    return g.to(torch.bfloat16) if dtype == GRAD_BF16 else g


def device_initial_weights(nparams, std=0.01, seed=MASTER_SEED, device="cuda"):
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    t = torch.empty(nparams, dtype=torch.float32, device=device)
    t.normal_(0.0, float(std), generator=gen)
    return t
