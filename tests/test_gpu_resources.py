"""Handles give back what they allocate: weights, state, staging slots, snapshot buffers on their
way to the host, weight versions, streams and events.  Device memory in use after many
create / use / destroy cycles must be what it was before them."""
import numpy as np
import pytest

from paper_1509_04210_b200 import synth

pytestmark = pytest.mark.gpu


def _cycle(rb, torch, N, lam, n, host_grads, dev_grads, slot, host_dst):
    c = lam // n
    ps = rb.ParameterServer(N, lam, n, 0.01, 0.9, 5e-4)
    ps.set_weights(dev_grads[0])
    ps.enable_views(lam + 1)
    for l in range(c):                                        # host-buffer path: staging slots, upload stream
        ps.push_host(host_grads[l % len(host_grads)], 0)
    assert ps.step() == 1
    assert ps.pull_host(host_dst) == 1                        # snapshot buffer, download stream
    ps.set_option(rb.OPT_PUSH_MODE, rb.PUSH_COPY)             # device copies into staging slots
    for l in range(c):
        ps.push(dev_grads[l % len(dev_grads)], 1)
    assert ps.step_pull_many([slot]) == 1
    ptr, ts = ps.pull_view(0)                                 # a weight version
    assert ts == 2 and ptr
    ps.set_option(rb.OPT_PUSH_MODE, rb.PUSH_BORROW)
    ps.set_option(rb.OPT_GRAD_DTYPE, rb.GRAD_BF16)            # frees the fp32 staging slots
    ps.set_option(rb.OPT_GRAD_DTYPE, rb.GRAD_F32)
    for l in range(c - 1):                                    # destroyed with gradients still queued
        ps.push_host(host_grads[l % len(host_grads)], 2)
    ps.sync()
    ps.close()


def test_create_use_destroy_cycles_leave_device_memory_as_it_was():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, lam, n = 1 << 20, 6, 2
    host_grads = [torch.from_numpy(synth.gradient(N, l, 0)).pin_memory() for l in range(3)]
    dev_grads = [g.cuda() for g in host_grads]
    slot = torch.empty(N, device="cuda")
    host_dst = torch.empty(N).pin_memory()
    _cycle(rb, torch, N, lam, n, host_grads, dev_grads, slot, host_dst)     # first use: module load, lazy set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(40):
        _cycle(rb, torch, N, lam, n, host_grads, dev_grads, slot, host_dst)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    # one cycle allocates about 60 MB (2 vectors, 7 versions, 3 + 3 staging slots, 1 snapshot buffer);
    # a leak of any one of them would cost 160 MB or more over 40 cycles
    assert free0 - free1 < (32 << 20), (free0, free1)
    assert np.isfinite(host_dst.numpy()).all()
