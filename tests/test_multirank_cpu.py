"""The multi-rank part of bench.py on CPU (gloo, world size 2): the path has no exchange
step, so ranks are replicas; what crosses ranks is only the max of the step times, and the
reported value is the sum over replicas of bytes / (slowest time)."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = bench.max_over_ranks(ms, world)
    value = bench.whole_job_value(4_000_000_000, world, slowest)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, slowest, value))


def test_max_over_ranks_and_whole_job_value_with_gloo():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in res:
        assert slowest == pytest.approx(15.0)
        assert value == pytest.approx(2 * 4.0 / 15.0e-3)      # GB/s of both replicas at the slowest rank's time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_value(2_000_000_000, 1, 1.0) == pytest.approx(2000.0)
    ab = bench.algorithmic_bytes(8, 32, 1000)
    assert ab["total"] == 4 * 8 * 1000 * (8 * 32 + 3 * 8 - 8)
    assert sum(bench.round_bytes(8, 32, 1000, k) for k in range(1, 39)) == ab["rounds"]
