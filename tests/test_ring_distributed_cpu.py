"""ring.DistributedRing driven on CPU by two gloo ranks.

There is one GPU at most where this runs, so the driver's logic (which peer buffer it
takes, where the barriers sit, how the counters of the fused form are wired between
neighbours, the epoch) is exercised with stand-ins: symmetric memory is a pair of
shared-memory CPU tensors, the stream barrier is dist.barrier(), and the plan's
rank-level calls are a few lines of torch on those tensors that follow the library's
own schedule (cerar_rank_round_slots).  The stand-in for the fused call runs the same
counter protocol as the kernel: poll local counters (bounded), store the tile into the
neighbour's slot, publish landed / freed.  The result must be the oracle's."""
import os
import socket
import sys
import time

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TILE = 8192


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class _FakeHandle:
    def __init__(self, bufs):
        self.bufs = bufs

    def get_buffer(self, rank, sizes, dtype, storage_offset=0):
        n = int(np.prod(sizes))
        return self.bufs[rank][storage_offset:storage_offset + n]

    def barrier(self, channel=0, timeout_ms=0):
        import torch.distributed as dist
        dist.barrier()


class _FakeSymmMem:
    """symm_mem.empty hands out this rank's pre-shared tensor of the requested size;
    rendezvous returns a handle that sees every rank's."""

    def __init__(self, rank, shared):
        self.rank, self.shared = rank, shared          # shared: {numel: [tensor of rank 0, tensor of rank 1]}

    def empty(self, n, dtype=None, device=None):
        return self.shared[(int(n), dtype)][self.rank]

    def rendezvous(self, t, group):
        for (n, dt), bufs in self.shared.items():
            if bufs[self.rank].data_ptr() == t.data_ptr():
                return _FakeHandle(bufs)
        raise AssertionError("rendezvous on a tensor that empty() did not hand out")


class _CpuPlan:
    """The rank-level calls on CPU tensors, slots from the library (host-only plan)."""

    def __init__(self, real_plan):
        self.real = real_plan
        self.N, self.c, self.L = real_plan.N, real_plan.c, real_plan.L
        self.calls = []

    def rank_workspace_bytes(self, d):
        return self.real.rank_workspace_bytes(d)

    def ring_tiles(self, d):
        return self.real.ring_tiles(d)

    def rank_round_slots(self, k):
        return self.real.rank_round_slots(k)

    def _rows(self, ws, d):
        return ws.view(self.c + self.N + 1, d // self.c)

    def rank_encode(self, rank, grad, ws, d, stream=0):
        import torch
        U = torch.from_numpy(self.real.get_U(rank)).float()
        self._rows(ws, d)[self.N + 1:self.N + 1 + self.c] = (grad.view(self.c, -1).T @ U).T
        self.calls.append(("encode", rank))

    def _message(self, W, k, q0, q1):
        prev, cancel, add, land = self.real.rank_round_slots(k)
        x = 0.0
        if prev >= 0:
            x = x + W[prev, q0:q1]
        if cancel >= 0:
            x = x - W[cancel, q0:q1]
        if add >= 0:
            x = x + W[add, q0:q1]
        return land, x

    def rank_round(self, rank, ws, peer_ws, d, k, stream=0):
        p = d // self.c
        land, x = self._message(self._rows(ws, d), k, 0, p)
        self._rows(peer_ws, d)[land] = x
        self.calls.append(("round", rank, k))

    def rank_round_msg(self, rank, ws, msg, d, k, stream=0):
        p = d // self.c
        _land, x = self._message(self._rows(ws, d), k, 0, p)
        msg.copy_(x)
        self.calls.append(("round_msg", rank, k))

    def rank_round_msg_bf16(self, rank, ws, msg, d, k, stream=0):
        import torch
        p = d // self.c
        _land, x = self._message(self._rows(ws, d), k, 0, p)
        msg.copy_(x.to(torch.bfloat16))                   # torch rounds to nearest, ties to even
        self.calls.append(("round_msg_bf16", rank, k))

    def rank_recv_bf16(self, rank, ws, msg, d, k, stream=0):
        import torch
        land = self.real.rank_round_slots(k)[3]
        self._rows(ws, d)[land] = msg.to(torch.float32)
        self.calls.append(("recv_bf16", rank, k))

    def rank_rounds_fused(self, rank, ws, peer_ws, landed_local, freed_local, landed_next, freed_prev, d, epoch,
                          stream=0):
        p = d // self.c
        nt = self.ring_tiles(d)
        base = epoch * (self.L + 1)
        W, Pw = self._rows(ws, d), self._rows(peer_ws, d)

        def wait(t, want):
            t0 = time.time()
            while int(t) < want:
                assert time.time() - t0 < 60, "a neighbour never answered"
                time.sleep(0.0005)

        for k in range(1, self.L + 1):
            for t in range(nt):
                if k >= 2:
                    wait(landed_local[t], base + k - 1)
                    wait(freed_local[t], base + k - 1)
                q0, q1 = t * TILE, min((t + 1) * TILE, p)
                land, x = self._message(W, k, q0, q1)
                Pw[land, q0:q1] = x
                landed_next[t] = base + k
                freed_prev[t] = base + k
        for t in range(nt):
            wait(landed_local[t], base + self.L)
        self.calls.append(("fused", rank, epoch))

    def rank_decode(self, rank, ws, out, d, scale=1.0, stream=0):
        import torch
        from paper_2609_23898_b200 import ring
        R = torch.from_numpy(self.real.get_R(rank)).float()
        Y = self._rows(ws, d)[ring.y_slots(self.real)]
        out.copy_((scale * (Y.T @ R)).T.reshape(-1))
        self.calls.append(("decode", rank))


def _worker(rank, world, port, c, p, shared, fused, q):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm_mem
    from oracle import designs as Dz
    from oracle import protocol as P
    from paper_2609_23898_b200 import cerar, ring
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, d = world, c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(5))
    plan = _CpuPlan(cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True))
    fake = _FakeSymmMem(rank, shared)
    symm_mem.empty, symm_mem.rendezvous = fake.empty, fake.rendezvous
    torch.cuda.current_device = lambda: 0
    real_device = torch.device
    torch.device = lambda *a, **k: real_device("cpu")
    r = ring.DistributedRing(plan, d)
    torch.device = real_device
    assert r.peer_ws.data_ptr() == shared[(plan.rank_workspace_bytes(d) // 4, torch.float32)][(rank + 1) % N].data_ptr()
    errs = []
    for rep in range(2):                                  # the second aggregation reuses buffers and counters
        rng = np.random.default_rng(100 + rep)
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(N)]
        out = torch.empty(d)
        r.allreduce(torch.from_numpy(grads[rank]), out, 0.5, 0, fused=fused)
        ora = P.allreduce([g.astype(np.float64) for g in grads], des.U, des.R, 0.5)
        errs.append(P.rel_l2(out.numpy(), ora["out"][rank]))
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, errs, r.epoch, [c_[0] for c_ in plan.calls]))


@pytest.mark.parametrize("fused", [False, True])
def test_distributed_ring_driver_with_two_gloo_ranks(fused):
    import torch
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    from oracle import designs as Dz
    from paper_2609_23898_b200 import cerar
    N, c, p = 2, 3, TILE + 100                            # two tiles, the second ragged
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(5))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True)
    n_ws, nt = plan.rank_workspace_bytes(d) // 4, plan.ring_tiles(d)
    assert nt == 2
    shared = {(n_ws, torch.float32): [torch.zeros(n_ws).share_memory_() for _ in range(N)],
              (2 * nt, torch.int32): [torch.zeros(2 * nt, dtype=torch.int32).share_memory_() for _ in range(N)]}
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, N, port, c, p, shared, fused, q)) for r in range(N)]
    for pr in procs:
        pr.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    L = c + N - 2
    for rank, errs, epoch, calls in res:
        assert max(errs) < 5e-6, errs
        if fused:
            assert epoch == 2 and calls == ["encode", "fused", "decode"] * 2
        else:
            assert calls == (["encode"] + ["round"] * L + ["decode"]) * 2


def _worker_sendrecv(rank, world, port, c, p, q, bf16=False):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    from oracle import designs as Dz
    from oracle import protocol as P
    from paper_2609_23898_b200 import cerar, ring
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, d = world, c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(6))
    plan = _CpuPlan(cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True))
    r = ring.SendRecvRing(plan, d, device=torch.device("cpu"), bf16_messages=bf16)
    errs = []
    for rep in range(2):
        rng = np.random.default_rng(300 + rep)
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(N)]
        out = torch.empty(d)
        r.allreduce(torch.from_numpy(grads[rank]), out, 1.0 / N, 0)
        ora = P.allreduce([g.astype(np.float64) for g in grads], des.U, des.R, 1.0 / N)
        errs.append(P.rel_l2(out.numpy(), ora["out"][rank]))
    dist.barrier()
    dist.destroy_process_group()
    q.put((rank, errs, [c_[0] for c_ in plan.calls]))


@pytest.mark.parametrize("N,c", [(2, 3), (3, 4)])
def test_send_receive_ring_driver_with_gloo_ranks(N, c):
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    p = 37
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker_sendrecv, args=(r, N, port, c, p, q)) for r in range(N)]
    for pr in procs:
        pr.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    L = c + N - 2
    for rank, errs, calls in res:
        assert max(errs) < 5e-6, errs
        assert calls == (["encode"] + ["round_msg"] * L + ["decode"]) * 2


def test_send_receive_ring_driver_with_bf16_messages():
    """The driver's bfloat16 transport: round on the sender, move 2-byte buffers, expand on the receiver
    (stand-ins for the two calls use torch's own bfloat16 conversion).  With orthogonal encoders the
    result is the exact mean up to the messages' 2^-8 rounding."""
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    N, c, p = 3, 4, 37
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker_sendrecv, args=(r, N, port, c, p, q, True)) for r in range(N)]
    for pr in procs:
        pr.start()
    res = sorted(q.get(timeout=240) for _ in procs)
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    L = c + N - 2
    for rank, errs, calls in res:
        assert 1e-5 < max(errs) < 2.0 ** -8 * (c + N), errs
        assert calls == (["encode"] + ["round_msg_bf16", "recv_bf16"] * L + ["decode"]) * 2

