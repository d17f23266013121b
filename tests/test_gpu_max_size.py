"""A vector longer than 2^32 weights: every index in the kernels and in the host code must be
64-bit.  The weights sampled span the whole vector (both ends, both sides of the 2^32 boundary and
random positions), and because weights never interact the oracle run on the sample alone is exact.
Covers the fused update (bf16 gradients, momentum and decay), pulls fused into the launch, a
stand-alone pull, the leaf averaging kernel and the state export."""
import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, REL_ONE_STEP, rel_err, to_host

pytestmark = pytest.mark.gpu

N_HUGE = (1 << 32) + (1 << 20) + 13        # ragged: not a multiple of 8, ends inside a tile


def _indices(N, seed):
    rng = np.random.default_rng(seed)
    edge = 1 << 32
    parts = [np.arange(96), np.arange(N - 96, N), np.arange(edge - 4200, edge + 4200),
             np.arange((1 << 31) - 64, (1 << 31) + 64), rng.integers(0, N, 6000)]
    return np.unique(np.concatenate(parts)).astype(np.int64)


def test_update_pull_and_leaf_average_beyond_four_giga_weights():
    import torch
    from paper_1509_04210_b200 import binding as rb

    torch.cuda.empty_cache()                                   # blocks cached by earlier tests count as free
    free, _ = torch.cuda.mem_get_info()
    need = N_HUGE * (4 + 4 + 4 + 4 + 4 + 2 * 3) + (2 << 30)   # weights, state, a temporary, slot, average, 3 bf16 gradients
    if free < need:
        pytest.skip("needs %.0f GB of free device memory, %.0f GB are free" % (need / 1e9, free / 1e9))
    N, lam, n = N_HUGE, 6, 2                                   # c = 3
    idx = _indices(N, 3)
    idx_d = torch.from_numpy(idx).cuda()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77)

    def normal(std, dtype):                                    # filled in pieces: no second full-size temporary
        out = torch.empty(N, dtype=dtype, device="cuda")
        piece = 1 << 28
        for lo in range(0, N, piece):
            hi = min(N, lo + piece)
            out[lo:hi] = (torch.randn(hi - lo, device="cuda", generator=gen) * std).to(dtype)
        return out

    th0 = normal(0.01, torch.float32)
    grads = [normal(1e-3, torch.bfloat16) for _ in range(3)]
    slot = torch.empty(N, dtype=torch.float32, device="cuda")
    ps = rb.ParameterServer(N, lam, n, 0.01, 0.9, 5e-4)
    ps.set_option(rb.OPT_GRAD_DTYPE, rb.GRAD_BF16)
    ps.set_weights(th0)
    o = ora.OraclePS(len(idx), lam, n, 0.01, 0.9, 5e-4)
    o.set_grad_dtype(ora.GRAD_BF16)
    o.set_weights(to_host(th0[idx_d]))
    del th0
    samples = [to_host(g[idx_d].view(torch.int16)).view(np.uint16) for g in grads]

    for upd in range(1, 4):
        for l in range(3):
            ps.push(grads[(l + upd) % 3], upd - 1)
            o.push(samples[(l + upd) % 3], upd - 1)
        # odd updates: the pull rides in the update's launch; even ones: a launch of its own
        if upd % 2:
            assert ps.step_pull_many([slot]) == 1
        else:
            assert ps.step() == 1
            assert ps.pull(slot) == upd
        assert o.step() == 1
        ps.sync()
        want = o.pull()[0]
        tol = REL_ONE_STEP if upd == 1 else REL_100_STEPS
        assert rel_err(to_host(slot[idx_d]), want) <= tol, upd
        assert ps.timestamp() == o.timestamp() == upd
    ps.export_state(None, slot)                                # the velocity, through the same buffer
    ps.sync()
    assert rel_err(to_host(slot[idx_d]), o.state()) <= REL_100_STEPS
    ps.close()

    # the server tree (Section 3.3) at the same length: a leaf averages the three vectors into a float
    # vector, the root takes the relayed average with its three timestamps
    avg = torch.empty(N, dtype=torch.float32, device="cuda")
    root = rb.ParameterServer(N, lam, n, 0.01, 0.9, 5e-4)
    th1 = normal(0.01, torch.float32)
    root.set_weights(th1)
    o2 = ora.OraclePS(len(idx), lam, n, 0.01, 0.9, 5e-4)
    o2.set_grad_dtype(ora.GRAD_BF16)
    o2.set_weights(to_host(th1[idx_d]))
    del th1
    rb.leaf_average(grads, rb.GRAD_BF16, N, avg)
    assert root.push_group([avg], [0, 0, 0]) == 3
    assert o2.push_relay(samples, [0, 0, 0]) == 3
    assert root.step() == 1 and o2.step() == 1
    assert root.pull(slot) == 1
    root.sync()
    assert rel_err(to_host(slot[idx_d]), o2.pull()[0]) <= REL_ONE_STEP
    np.testing.assert_array_equal(root.last_messages()["step"].view(np.uint32), o2.last_messages()["step"].view(np.uint32))
    root.close()
    del avg, slot, grads
    torch.cuda.empty_cache()                                   # give the 100 GB back before the next test
