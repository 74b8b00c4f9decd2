"""The multi-GPU mode is replicas only: ranks share nothing but the timing reduction.
Two CPU processes over gloo check that reduction (max over ranks, whole-job time per token)."""

import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 0.40 + 0.05 * rank                      # rank 1 is the slower replica
    worst, us_token = bench.aggregate_replicas(ms, world, dist, "cpu")
    out.put((rank, worst, us_token))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 500
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, us_token in got:
        assert worst == pytest.approx(0.45)               # max over ranks, on every rank
        assert us_token == pytest.approx(225.0)           # 0.45 ms for two tokens


def test_one_replica_is_the_identity():
    import bench
    assert bench.aggregate_replicas(0.5, 1, None, "cpu") == (0.5, 500.0)
