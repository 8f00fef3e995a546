"""One worker per rank, checked without a GPU.

The library tells which slots of the per-worker layout a round reads and where the
message lands (cerar_rank_round_slots).  Here (a) the schedule's hazards are checked
by reading it, and (b) two gloo ranks play the two workers of an N = 2 ring with a
few lines of numpy each, moving the messages with torch.distributed, and must end
with what the oracle computes for the whole ring.  The numpy steps here are test
code: the product path for this is the rank-level CUDA kernels."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _plan(N, c, seed=0):
    from oracle import designs as Dz
    from paper_2609_23898_b200 import cerar
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(seed))
    return des, cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True)


@pytest.mark.parametrize("N,c", [(2, 2), (2, 5), (4, 8), (5, 9), (8, 32), (16, 16)])
def test_schedule_has_no_same_round_hazard_and_fills_y_in_order(N, c):
    from paper_2609_23898_b200 import ring
    des, plan = _plan(N, c)
    L = c + N - 2
    sched = ring.round_schedule(plan)
    assert [s[0] for s in sched] == list(range(1, L + 1))
    rows = c + N + 1
    assert plan.rank_workspace_bytes(c * 10) == 4 * rows * 10
    # what each slot holds, per worker (all workers alike): ("delta", j) or ("y", m)
    holds = {N + j: ("delta", j) for j in range(1, c + 1)}
    for k, prev, cancel, add, land in sched:
        reads = [s for s in (prev, cancel, add) if s >= 0]
        assert land not in reads                  # the neighbour writes `land` while the owner reads `reads`
        assert 0 <= land < rows and all(0 <= s < rows for s in reads)
        assert (prev >= 0) == (k >= 2) and (cancel >= 0) == (k > N) and (add >= 0) == (k <= c)
        if prev >= 0:
            assert holds[prev] == ("y", k - 1)
        if cancel >= 0:
            assert holds[cancel] == ("delta", k - N)
        if add >= 0:
            assert holds[add] == ("delta", k)
        # the landing slot is free: never written, or a delta that was cancelled in an EARLIER round
        if land in holds:
            kind, j = holds[land]
            assert kind == "delta" and j + N < k
        holds[land] = ("y", k)
    ys = ring.y_slots(plan)
    assert len(ys) == L + 1
    assert [holds[s] for s in ys[:L]] == [("y", m) for m in range(1, L + 1)]
    assert holds[ys[L]] == ("delta", c)           # y_{L+1} = delta_c (Sec. II-A)
    with pytest.raises(Exception):
        plan.rank_round_slots(0)
    with pytest.raises(Exception):
        plan.rank_round_slots(L + 1)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, c, p, q):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    from oracle import protocol as P
    from paper_2609_23898_b200 import ring
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N = world
    des, plan = _plan(N, c, seed=7)
    rng = np.random.default_rng(11)
    grads = [rng.standard_normal(c * p) for _ in range(N)]        # every rank draws all, keeps its own
    U, R = plan.get_U(rank), plan.get_R(rank)
    ws = np.full((c + N + 1, p), np.nan)
    ws[N + 1:N + 1 + c] = (grads[rank].reshape(c, p).T @ U).T     # slot N+j = delta_j
    nxt, prv = (rank + 1) % N, (rank - 1) % N
    for k, prev, cancel, add, land in ring.round_schedule(plan):
        x = np.zeros(p)
        if prev >= 0:
            x = x + ws[prev]
        if cancel >= 0:
            x = x - ws[cancel]
        if add >= 0:
            x = x + ws[add]
        recv = torch.empty(p, dtype=torch.float64)
        reqs = [dist.isend(torch.from_numpy(x.copy()), nxt), dist.irecv(recv, prv)]
        for r in reqs:
            r.wait()
        ws[land] = recv.numpy()
        dist.barrier()
    Y = ws[ring.y_slots(plan)]                                       # (L+1, p)
    out = (Y.T @ R).T.reshape(-1)
    ora = P.allreduce(grads, des.U, des.R, 1.0)
    err = P.rel_l2(out, ora["out"][rank])
    err_y = P.rel_l2(Y, ora["Y"][rank].T)
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, err, err_y))


@pytest.mark.parametrize("c", [2, 5])
def test_two_gloo_ranks_run_the_ring_and_match_the_oracle(c):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, c, 6, q)) for r in range(2)]
    for pr in procs:
        pr.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    for _, err, err_y in res:
        assert err_y < 1e-12 and err < 1e-12
