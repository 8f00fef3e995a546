"""CERAR with one worker per rank: drivers around the cerar_rank_* calls.

The protocol (Sec. II, Algorithm 1) per worker i: encode, then L rounds in which the
worker forms message k from its own slots and stores it into the landing slot of
worker i+1, then decode.  The kernels are the library's; this module only owns the
buffers and the order of the calls.

LocalRing         all N workers in this process on one GPU, each with its own
                  workspace; "the neighbour's memory" is just another tensor and
                  stream order stands in for the barrier between rounds.  This is
                  what the GPU tests and the single-GPU measurements run.
DistributedRing   one worker per process and GPU (torch.distributed, NCCL): the
                  workspace lives in symmetric memory, the neighbour's copy is a
                  peer-mapped tensor, and either a device-side barrier on the stream
                  separates the rounds or (fused=True) one kernel runs all rounds
                  and orders itself against the neighbours tile by tile through
                  counters in symmetric memory.  Needs N GPUs with peer access.
SendRecvRing      one worker per process without peer access (the paper's own setting:
                  GPUs on PCIe, one process each): the message of a round is formed in a
                  local buffer and moved by a batched send / receive pair of
                  torch.distributed (NCCL between GPUs), received straight into the
                  landing slot of the workspace.
"""
from __future__ import annotations

from . import cerar


def round_schedule(plan):
    """[(k, slot_prev, slot_cancel, slot_add, slot_land)] for k = 1..L as the library
    computes them (-1 = the term is absent in that round)."""
    return [(k,) + plan.rank_round_slots(k) for k in range(1, plan.L + 1)]


def y_slots(plan):
    """Slots that hold y_1 .. y_{L+1} after round L (the rows decode reads, in order)."""
    return list(range(plan.L)) + [plan.N + plan.c]


class LocalRing:
    def __init__(self, plan, d: int, device="cuda"):
        import torch
        if d % plan.c:
            raise ValueError("d must be a multiple of c")
        self.plan, self.d, self.p = plan, d, d // plan.c
        self.N, self.c, self.L = plan.N, plan.c, plan.L
        n = plan.rank_workspace_bytes(d) // 4
        self.ws = [torch.empty(n, dtype=torch.float32, device=device) for _ in range(self.N)]
        # tile counters of the fused rounds: [worker][landed | freed][tile], zero once, never reset
        self.counters = torch.zeros(2 * self.N * plan.ring_tiles(d), dtype=torch.int32, device=device)
        self.epoch = 0

    def grad_view(self, i):
        """The D rows of worker i's workspace as a length-d tensor (in-place use)."""
        o = (self.N + 1) * self.p
        return self.ws[i][o:o + self.d]

    def encode(self, grads, stream=0):
        for i in range(self.N):
            self.plan.rank_encode(i, grads[i], self.ws[i], self.d, stream)

    def round(self, k, stream=0):
        # every worker's launch of round k is queued after all launches of round k-1
        for i in range(self.N):
            self.plan.rank_round(i, self.ws[i], self.ws[(i + 1) % self.N], self.d, k, stream)

    def rounds_fused(self, stream=0):
        """All L rounds of all N workers in one cooperative launch, ordered per tile by counters."""
        self.plan.ring_rounds_fused_local(self.ws, self.counters, self.d, self.epoch, stream)
        self.epoch += 1

    def decode(self, outs, scale=1.0, stream=0):
        for i in range(self.N):
            self.plan.rank_decode(i, self.ws[i], outs[i], self.d, scale, stream)

    def allreduce(self, grads, outs, scale=1.0, stream=0, fused=False):
        self.encode(grads, stream)
        if fused:
            self.rounds_fused(stream)
        else:
            for k in range(1, self.L + 1):
                self.round(k, stream)
        self.decode(outs, scale, stream)


class DistributedRing:
    """One worker per rank.  `group` is a torch.distributed process group of exactly
    plan.N ranks whose devices have peer access to one another."""

    def __init__(self, plan, d: int, group=None, device=None):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        group = group if group is not None else dist.group.WORLD
        self.rank, world = dist.get_rank(group), dist.get_world_size(group)
        if world != plan.N:
            raise ValueError(f"the plan is for N={plan.N} workers, the group has {world} ranks")
        if d % plan.c:
            raise ValueError("d must be a multiple of c")
        self.plan, self.d, self.p = plan, d, d // plan.c
        self.N, self.c, self.L = plan.N, plan.c, plan.L
        n = plan.rank_workspace_bytes(d) // 4
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.ws = symm_mem.empty(n, dtype=torch.float32, device=dev)
        self._hdl = symm_mem.rendezvous(self.ws, group)
        self.peer_ws = self._hdl.get_buffer((self.rank + 1) % self.N, (n,), torch.float32)
        self.barrier_timeout_ms = 10000
        # tile counters of the fused rounds, [landed | freed][tile], in symmetric memory as well
        nt = plan.ring_tiles(d)
        self.counters = symm_mem.empty(2 * nt, dtype=torch.int32, device=self.ws.device)
        self.counters.zero_()
        self._chdl = symm_mem.rendezvous(self.counters, group)
        nxt, prv = (self.rank + 1) % self.N, (self.rank - 1) % self.N
        self._landed_next = self._chdl.get_buffer(nxt, (nt,), torch.int32, 0)
        self._freed_prev = self._chdl.get_buffer(prv, (nt,), torch.int32, nt)
        self._nt = nt
        self.epoch = 0

    def _barrier(self):
        # on the current stream: all kernels of the round before, on every rank, are
        # complete and visible before anything after it starts
        self._hdl.barrier(channel=0, timeout_ms=self.barrier_timeout_ms)

    def allreduce(self, grad, out, scale=1.0, stream=0, fused=False):
        """grad, out: this rank's length-d device tensors; `stream` must be torch's current stream.
        fused=True: one kernel for all rounds, ordered against the neighbours per tile by counters
        in symmetric memory, instead of one kernel and one barrier per round."""
        self._barrier()                      # the neighbours are done reading the previous call's slots
        self.plan.rank_encode(self.rank, grad, self.ws, self.d, stream)
        if fused:
            # no further barrier: a message only ever lands in a slot whose owner has either not used
            # it yet in this aggregation (slots 0..N) or has reported its last read of it (`freed`)
            self.plan.rank_rounds_fused(self.rank, self.ws, self.peer_ws, self.counters,
                                        self.counters[self._nt:], self._landed_next, self._freed_prev,
                                        self.d, self.epoch, stream)
            self.epoch += 1
        else:
            for k in range(1, self.L + 1):
                self.plan.rank_round(self.rank, self.ws, self.peer_ws, self.d, k, stream)
                self._barrier()
        self.plan.rank_decode(self.rank, self.ws, out, self.d, scale, stream)


class SendRecvRing:
    """One worker per rank, messages moved by torch.distributed send / receive.
    bf16_messages=True: the sender rounds every message to bfloat16 and the receiver expands it
    (cerar_rank_round_msg_bf16 / cerar_rank_recv_bf16): half the bytes on the wire; fp8_messages=True:
    e4m3 codes with a power-of-two scale per 1024 positions (cerar_rank_round_msg_fp8 /
    cerar_rank_recv_fp8): a quarter.  Both for well-conditioned designs only."""

    def __init__(self, plan, d: int, group=None, device=None, bf16_messages=False, fp8_messages=False):
        import torch
        import torch.distributed as dist
        self.group = group if group is not None else dist.group.WORLD
        self.rank, world = dist.get_rank(self.group), dist.get_world_size(self.group)
        if world != plan.N:
            raise ValueError(f"the plan is for N={plan.N} workers, the group has {world} ranks")
        if d % plan.c:
            raise ValueError("d must be a multiple of c")
        self.plan, self.d, self.p = plan, d, d // plan.c
        self.N, self.c, self.L = plan.N, plan.c, plan.L
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.ws = torch.empty(plan.rank_workspace_bytes(d) // 4, dtype=torch.float32, device=dev)
        self.bf16 = bool(bf16_messages)
        self.fp8 = bool(fp8_messages)
        if self.bf16 and self.fp8:
            raise ValueError("one message format at a time")
        if self.fp8:
            # e4m3 codes plus one scale per tile (cerar_rank_round_msg_fp8 / cerar_rank_recv_fp8)
            nb = (plan.fp8_message_bytes(d) + 15) // 16 * 16
            self.msg = torch.empty(nb, dtype=torch.uint8, device=dev)
            self.msg_in = torch.empty(nb, dtype=torch.uint8, device=dev)
        else:
            self.msg = torch.empty(self.p, dtype=torch.bfloat16 if self.bf16 else torch.float32, device=dev)
            self.msg_in = torch.empty(self.p, dtype=torch.bfloat16, device=dev) if self.bf16 else None
        self.schedule = round_schedule(plan)
        self.nxt = dist.get_global_rank(self.group, (self.rank + 1) % self.N)
        self.prv = dist.get_global_rank(self.group, (self.rank - 1) % self.N)

    def allreduce(self, grad, out, scale=1.0, stream=0):
        """grad, out: this rank's length-d tensors; `stream` must be torch's current stream (the
        send and the receive are ordered against it by torch.distributed)."""
        import torch.distributed as dist
        self.plan.rank_encode(self.rank, grad, self.ws, self.d, stream)
        rows = self.ws.view(self.c + self.N + 1, self.p)
        for k, _prev, _cancel, _add, land in self.schedule:
            if self.fp8:
                self.plan.rank_round_msg_fp8(self.rank, self.ws, self.msg, self.d, k, stream)
            elif self.bf16:
                self.plan.rank_round_msg_bf16(self.rank, self.ws, self.msg, self.d, k, stream)
            else:
                self.plan.rank_round_msg(self.rank, self.ws, self.msg, self.d, k, stream)
            ops = [dist.P2POp(dist.isend, self.msg, self.nxt, self.group),
                   dist.P2POp(dist.irecv, self.msg_in if (self.bf16 or self.fp8) else rows[land], self.prv, self.group)]
            for req in dist.batch_isend_irecv(ops):
                req.wait()
            if self.fp8:
                self.plan.rank_recv_fp8(self.rank, self.ws, self.msg_in, self.d, k, stream)
            elif self.bf16:
                self.plan.rank_recv_bf16(self.rank, self.ws, self.msg_in, self.d, k, stream)
        self.plan.rank_decode(self.rank, self.ws, out, self.d, scale, stream)
