"""The range-sharding plumbing over the real CUDA server, on the one GPU a run has: a process
group of one rank (NCCL), so that every device-side step of `sharding.ShardedServer` -- range
slices of a device gradient, the per-rank server's push / step / pull on device tensors, the
gathered pull, the single-timestamp check -- runs on the GPU and is compared with the oracle.
The two-rank exchange itself is covered on CPU (gloo) in test_dist_gloo.py."""
import os
import socket

import numpy as np
import pytest

from oracle import rudra_oracle as ora
from paper_1509_04210_b200 import synth

from helpers import REL_100_STEPS, rel_err, to_device, to_host

pytestmark = pytest.mark.gpu


def test_sharded_server_of_one_rank_on_the_gpu_equals_the_oracle():
    import torch
    import torch.distributed as dist
    from paper_1509_04210_b200 import binding as rb
    from paper_1509_04210_b200 import sharding

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        N, lam, n, a0, m, wd = 300011, 6, 2, 0.05, 0.9, 5e-4
        empty = lambda k, kind: torch.empty(k, dtype=torch.float32, device="cuda")
        srv = sharding.ShardedServer(lambda k: rb.ParameterServer(k, lam, n, a0, m, wd), N, lam // n, empty)
        assert srv.bounds == [(0, N)]
        cpu = ora.OraclePS(N, lam, n, a0, m, wd)
        th0 = synth.initial_weights(N, 0.01, 5)
        srv.set_weights(to_device(th0))
        cpu.set_weights(th0)
        sched = rb.Scheduler(lam, n, rb.SCHED_SOFTSYNC_ROUNDS, 11)
        full = torch.empty(N, device="cuda")
        updates = 0
        for _ in range(300):
            e = sched.next(1)[0]
            kind, l = int(e["kind"]), int(e["learner"])
            if kind == rb.EV_PUSH:
                g = synth.gradient(N, l, int(e["seq"]), 1e-2)
                srv.push(0, to_device(g), int(e["pulled_ts"]))
                cpu.push(g, int(e["pulled_ts"]))
            elif kind == rb.EV_STEP:
                assert srv.step() == 1 and cpu.step() == 1
                updates += 1
                assert srv.check_single_timestamp() == int(e["ts"]) == cpu.timestamp()
            elif kind == rb.EV_PULL:
                assert srv.pull(full) == int(e["ts"])
                torch.cuda.synchronize()
                assert rel_err(to_host(full), cpu.pull()[0]) <= REL_100_STEPS
        assert updates > 20
        srv.server.close()
    finally:
        dist.destroy_process_group()
