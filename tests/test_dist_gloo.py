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
