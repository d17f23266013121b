"""The benchmark's bandwidth probe (librudra_probe.so, a library of its own outside the
parameter-server interface): it must move exactly the vectors it is given."""
import numpy as np
import pytest

from helpers import to_host

pytestmark = pytest.mark.gpu


def test_stream_probe_reads_and_writes_what_it_is_given():
    # the measurement utility: every destination receives 1 + 0.5 * (sum of the sources), canaries intact
    import torch
    from paper_1509_04210_b200 import probe as rb

    N = 8 * 256 * 5 + 8 * 17
    srcs = [torch.full((N,), float(i + 1), device="cuda") for i in range(5)]
    big = [torch.full((N + 16,), -7.0, device="cuda") for _ in range(3)]
    dsts = [b[8:8 + N] for b in big]
    assert rb.stream_probe(srcs, dsts, N) == 0
    torch.cuda.synchronize()
    for b in big:
        h = to_host(b)
        assert np.all(h[8:8 + N] == 1.0 + 0.5 * 15.0) and np.all(h[:8] == -7.0) and np.all(h[8 + N:] == -7.0)
    assert rb.stream_probe(srcs, [], N) == 0 and rb.stream_probe([], dsts, N) == 0
    torch.cuda.synchronize()
    assert np.all(to_host(dsts[0]) == 1.0)
    with pytest.raises(RuntimeError):
        rb.stream_probe(srcs * 13, dsts, N)            # 65 sources: more than the table holds
    with pytest.raises(RuntimeError):
        rb.stream_probe([srcs[0][1:]], dsts, N - 8)    # misaligned source
