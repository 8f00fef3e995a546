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


def _ring_worker(rank, world, port, c, p, shared, q):
    """bench.ring_block (the N > 1 part of the benchmark: one worker per rank) driven on CPU: gloo
    ranks, shared-memory tensors in place of symmetric memory, torch stand-ins for the rank-level
    library calls (the stand-ins of tests/test_ring_distributed_cpu.py)."""
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm_mem
    import bench
    from paper_2609_23898_b200 import cerar, inputs
    from tests.test_ring_distributed_cpu import _CpuPlan, _FakeSymmMem
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N = world
    real = cerar.Plan.create(N, c, cerar.EPSILON, 1e-3, B=inputs.base_matrix(N, c, 0), host_only=True)
    plan = _CpuPlan(real)
    fake = _FakeSymmMem(rank, shared)
    symm_mem.empty, symm_mem.rendezvous = fake.empty, fake.rendezvous
    block = bench.ring_block(world, rank, torch.device("cpu"), plan=plan, d=c * p, reps=2)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, block, [x[0] for x in plan.calls]))


def test_ring_block_of_the_benchmark_with_two_gloo_ranks():
    import torch
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    from paper_2609_23898_b200 import cerar, inputs
    N, c, p = 2, 2, 8192 + 100                           # c = N: the design reproduces the mean to O(eps)
    d = c * p
    plan = cerar.Plan.create(N, c, cerar.EPSILON, 1e-3, B=inputs.base_matrix(N, c, 0), host_only=True)
    n_ws, nt = plan.rank_workspace_bytes(d) // 4, plan.ring_tiles(d)
    shared = {(n_ws, torch.float32): [torch.zeros(n_ws).share_memory_() for _ in range(N)],
              (2 * nt, torch.int32): [torch.zeros(2 * nt, dtype=torch.int32).share_memory_() for _ in range(N)]}
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_ring_worker, args=(r, N, port, c, p, shared, q)) for r in range(N)]
    for pr in procs:
        pr.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    L = c + N - 2
    for rank, block, calls in res:
        assert block["workers"] == N and block["c"] == c and block["L"] == L and block["d"] == d
        assert block["bytes_over_the_link_per_rank"] == 4 * p * L
        assert block["all_reduce_ms"] > 0
        for form in ("sendrecv", "peer_round_by_round", "peer_fused_rounds"):
            assert "error" not in block[form], block[form]
            assert block[form]["ms_per_aggregation"] > 0
            assert block[form]["ratio_to_all_reduce"] == pytest.approx(
                block[form]["ms_per_aggregation"] / block["all_reduce_ms"])
        assert block["identical_results"] is True
        assert block["rel_l2_vs_all_reduce_mean"] < 0.05
        assert block["status"].startswith("unmeasured")
        # warm-up + 2 timed aggregations per form, each through the driver's own order of calls
        assert calls.count("encode") == 9 and calls.count("decode") == 9
        assert calls.count("round_msg") == 3 * L and calls.count("round") == 3 * L and calls.count("fused") == 3
