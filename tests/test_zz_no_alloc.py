"""The no-allocation entry point against the regular host-buffer path, through the C interface.

rudra_ps_update_host_noalloc serves callers that cannot allocate device memory while running
(their own pool owns the GPU, or an allocation's device-wide synchronisation is not acceptable):
it stages gradients in a fixed array inside the library instead of buffers allocated on demand.
The update it performs must equal what rudra_ps_push_host + rudra_ps_step produce from the same
host gradients and step sizes, on two calls in a row (the second re-uses the shared array).
This file sorts last so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest

from paper_1509_04210_b200 import synth

from helpers import REL_ONE_STEP, rel_err

pytestmark = pytest.mark.gpu


def test_no_alloc_update_matches_push_host_and_step_twice():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N, c, m, wd = 100003, 3, 0.9, 5e-4
    th0 = synth.initial_weights(N, 0.01, 77)
    ps = rb.ParameterServer(N, c, 1, 0.05, m, wd)
    ps.set_option(rb.OPT_LR_POLICY, rb.LR_PER_GRADIENT)
    ps.set_weights_host(np.ascontiguousarray(th0))
    for warm in range(2):                                    # raise the timestamp so staleness can vary
        for l in range(c):
            ps.push_host(synth.gradient(N, l, 10 + warm, 1e-2, seed=5), ps.timestamp())
        assert ps.step() == 1
    theta = torch.empty(N, device="cuda")
    state = torch.empty(N, device="cuda")
    ps.export_state(theta, state)
    ps.sync()
    want_th = torch.empty(N, device="cuda")
    want_st = torch.empty(N, device="cuda")
    for call in range(2):
        grads = [synth.gradient(N, l, call, 1e-2, seed=5) for l in range(c)]
        ts = ps.timestamp()
        for g, back in zip(grads, (0, 2, 1)):                # staleness 0, 2, 1: three different step sizes
            ps.push_host(g, ts - back)
        assert ps.step() == 1
        assert list(ps.last_clock()["sigma"]) == [0, 2, 1]
        scales = ps.last_clock()["scale"]
        ps.export_state(want_th, want_st)
        ps.sync()
        assert rb.update_host_noalloc(theta, state, N, grads, scales, m, wd) == 0
        torch.cuda.synchronize()
        e_th = rel_err(theta.cpu().numpy(), want_th.cpu().numpy())
        e_st = rel_err(state.cpu().numpy(), want_st.cpu().numpy())
        assert e_th <= REL_ONE_STEP and e_st <= REL_ONE_STEP, (call, e_th, e_st)
    ps.close()


def test_no_alloc_rejects_what_does_not_fit():
    import torch
    from paper_1509_04210_b200 import binding as rb

    N = rb.NOALLOC_MAX_FLOATS // 2 + 64
    theta = torch.zeros(N, device="cuda")
    g = np.zeros(N, dtype=np.float32)
    with pytest.raises(rb.RudraError) as e:
        rb.update_host_noalloc(theta, None, N, [g, g], [0.1, 0.1], 0.0, 0.0)
    assert e.value.code == rb.E_INVAL and "does not fit" in str(e.value)
    with pytest.raises(rb.RudraError):
        rb.update_host_noalloc(theta, None, 64, [g], [0.1], 0.9, 0.0)   # momentum needs a state vector
    torch.cuda.synchronize()
    assert float(theta.abs().max()) == 0.0
