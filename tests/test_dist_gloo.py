"""The N > 1 host logic on two gloo ranks (CPU): barrier + max-over-ranks timing of independent
replicas, whole-job rate, per-rank seeds, and the reference arm's rank-0-only rule."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1509_04210_b200 import replicas, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.rank_info() == (rank, rank, world)
    dist.barrier()
    mine = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]
    got = replicas.max_over_ranks(mine)
    seed = replicas.replica_seed(synth.MASTER_SEED, rank)
    g = synth.gradient(64, 0, 0, seed=seed)
    out.put((rank, got, seed, float(g[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, seed, g0 in res:
        assert got == [15.0, 3.0, 7.0]
    assert res[0][2] != res[1][2] and res[0][3] != res[1][3]     # distinct streams per replica
    assert replicas.whole_job_rate(200, 2, 100.0) == 4000.0


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.rank_info()[2] >= 1


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "3", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


# ------------------------------------------------------------------------------------------------
# range sharding: host logic on two gloo ranks, the oracle standing in for the per-rank server
# ------------------------------------------------------------------------------------------------
class _OracleShard:
    """The per-rank server interface over the CPU oracle (torch CPU tensors in, numpy inside)."""

    def __init__(self, nparams, lam, n, a0, m, wd):
        from oracle import rudra_oracle as ora

        self.o = ora.OraclePS(nparams, lam, n, a0, m, wd)

    def set_weights(self, t):
        self.o.set_weights(t.numpy())

    def push(self, t, pulled_ts):
        return self.o.push(t.numpy(), pulled_ts)

    def step(self):
        return self.o.step()

    def pull(self, dst):
        w, ts = self.o.pull()
        dst.copy_(torch.from_numpy(w))
        return ts

    def timestamp(self):
        return self.o.timestamp()


def _shard_worker(rank, world, port, out):
    import numpy as np

    from oracle import rudra_oracle as ora
    from paper_1509_04210_b200 import binding as rb
    from paper_1509_04210_b200 import sharding

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, lam, n, a0, m, wd = 1000 + 37, 6, 2, 0.05, 0.9, 5e-4
    empty = lambda k, kind: torch.empty(k, dtype=torch.float32)
    srv = sharding.ShardedServer(lambda k: _OracleShard(k, lam, n, a0, m, wd), N, lam // n, empty)
    whole = ora.OraclePS(N, lam, n, a0, m, wd)            # the unsharded server, replayed on every rank
    th0 = synth.initial_weights(N, 0.01, 5)
    srv.set_weights(torch.from_numpy(th0))
    whole.set_weights(th0)
    sched = rb.Scheduler(lam, n, rb.SCHED_SOFTSYNC_ROUNDS, 11)     # same seed everywhere: one global order
    full = torch.empty(N)
    stamps = []
    for _ in range(400):
        e = sched.next(1)[0]
        kind, l = int(e["kind"]), int(e["learner"])
        if kind == rb.EV_PUSH:
            home = l % world                                # the learner lives on this rank
            g = synth.gradient(N, l, int(e["seq"]), 1e-2)
            srv.push(home, torch.from_numpy(g) if rank == home else None, int(e["pulled_ts"]))
            whole.push(g, int(e["pulled_ts"]))
        elif kind == rb.EV_STEP:
            assert srv.step() == 1 and whole.step() == 1
            assert srv.check_single_timestamp() == int(e["ts"]) == whole.timestamp()
            stamps.append(srv.timestamp())
        elif kind == rb.EV_PULL:
            assert srv.pull(full) == int(e["ts"])
            np.testing.assert_array_equal(full.numpy(), whole.pull()[0])    # ranges of one version, bit for bit
    out.put((rank, srv.bounds, stamps[-1], len(stamps)))
    dist.barrier()
    dist.destroy_process_group()


def test_range_sharded_server_keeps_one_timestamp_and_equals_the_whole():
    from paper_1509_04210_b200 import sharding

    for N, world in [(60965224, 8), (1037, 2), (100, 3), (63, 4), (1, 2)]:
        b = sharding.shard_bounds(N, world)
        assert b[0][0] == 0 and b[-1][1] == N and all(b[i][1] == b[i + 1][0] for i in range(world - 1))
        assert all(lo % sharding.ALIGN == 0 and hi >= lo for lo, hi in b)
    sizes = [hi - lo for lo, hi in sharding.shard_bounds(60965224, 8)]
    assert max(sizes) - min(sizes) <= sharding.ALIGN * 2
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == [(0, 512), (512, 1037)]
    assert res[0][2:] == res[1][2:] and res[0][3] > 30            # same timestamp history on both ranks
