"""One worker per rank on the GPU: the rank-level kernels (one launch per worker and
step, separate workspaces, the message stored through a pointer into the
neighbour's workspace) against the oracle, stage by stage, and against the
all-workers-per-launch pipeline (bit for bit wherever the order of operations is the same)."""
import numpy as np
import pytest

from oracle import designs as Dz
from tests._harness import rel_l2, run_library, run_oracle

pytestmark = pytest.mark.gpu

STAGE_TOL = 2e-6


@pytest.fixture(scope="module")
def mods():
    import torch
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    from paper_2609_23898_b200 import cerar, inputs, ring
    return cerar, inputs, ring


# FMA kernels (vector and scalar paths), both tensor-core tilings, N = 2, c = N
SHAPES = [(4, 8, 8192 + 260), (3, 5, 1031), (2, 2, 4), (4, 4, 4096), (8, 20, 2052),
          (8, 32, 4100), (8, 40, 1028), (4, 96, 388), (16, 16, 1028)]


@pytest.mark.parametrize("N,c,p", SHAPES)
@pytest.mark.parametrize("inplace", [False, True])
def test_local_ring_matches_oracle_and_batched_pipeline(mods, N, c, p, inplace):
    import torch
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(10 * N + c))
    g = inputs.gradients_numpy(N, d, "normal", seed=4)
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    ora = run_oracle(des.U, des.R, g, 0.5)
    s = torch.cuda.current_stream().cuda_stream
    r = ring.LocalRing(plan, d)
    for w in r.ws:
        w.fill_(float("nan"))
    if inplace:
        grads = [r.grad_view(i) for i in range(N)]
        for i in range(N):
            grads[i].copy_(torch.from_numpy(g[i]))
        outs = grads
    else:
        grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
        outs = [torch.full((d,), float("nan"), device="cuda") for _ in range(N)]
    r.encode(grads, s)
    rows = c + N + 1
    delta = np.stack([r.ws[i].view(rows, p)[N + 1:N + 1 + c].cpu().numpy() for i in range(N)])
    assert rel_l2(delta, ora["Delta_rows"]) < STAGE_TOL
    for k in range(1, plan.L + 1):
        r.round(k, s)
    ys = ring.y_slots(plan)
    Y = np.stack([r.ws[i].view(rows, p)[ys].cpu().numpy() for i in range(N)])
    assert rel_l2(Y, ora["Y_rows"]) < STAGE_TOL
    r.decode(outs, 0.5, s)
    torch.cuda.synchronize()
    plan.device_status(s)
    out = np.stack([o.cpu().numpy() for o in outs])
    assert max(rel_l2(out[i], ora["out"][i]) for i in range(N)) < 5e-6
    # same kernels, same order of operations as the all-workers-per-launch pipeline
    ref = run_library(cerar.Plan.create_custom(N, c, des.U, des.R), g, 0.5)
    assert np.array_equal(delta, ref["Delta"])
    assert np.array_equal(Y, ref["Y"])
    if c < 24:
        assert np.array_equal(out, ref["out"])
    else:
        # tensor-core decode: the two spent rows shift which inputs share a K = 8 product, and the
        # sum inside one product is not taken in row order
        assert rel_l2(out, ref["out"]) < 2e-6


def test_one_call_form_and_argument_checks(mods):
    import torch
    cerar, inputs, ring = mods
    N, c, p = 4, 8, 2048
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(2))
    g = inputs.gradients_numpy(N, d, "normal", seed=6)
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    ora = run_oracle(des.U, des.R, g, 1.0 / N)
    s = torch.cuda.current_stream().cuda_stream
    r = ring.LocalRing(plan, d)
    grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    for _ in range(2):                         # a second aggregation reuses the workspaces
        r.allreduce(grads, outs, 1.0 / N, s)
    torch.cuda.synchronize()
    assert max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N)) < 5e-6
    with pytest.raises(cerar.CerarError):
        plan.rank_round(0, r.ws[0], r.ws[0], d, 1, s)          # a worker is not its own neighbour
    with pytest.raises(cerar.CerarError):
        plan.rank_round(N, r.ws[0], r.ws[1], d, 1, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_round(0, r.ws[0], r.ws[1], d, plan.L + 1, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_encode(-1, grads[0], r.ws[0], d, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_decode(0, r.ws[0], outs[0], d + 1, 1.0, s)
    assert plan.rank_workspace_bytes(d) == 4 * (c + N + 1) * p


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 * 3 + 260), (8, 32, 8192 * 5 + 4), (2, 2, 8192 + 8), (3, 5, 20001),
                                   (16, 16, 8192 * 2), (5, 9, 7)])
def test_fused_rounds_one_launch_equals_round_by_round(mods, N, c, p):
    """All L rounds of all workers in one cooperative launch, ordered per tile by counters:
    same slots bit for bit as one launch per worker and round; several aggregations on the
    same counters (the epoch moves on, nothing is reset)."""
    import torch
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(3 * N + c))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    s = torch.cuda.current_stream().cuda_stream
    ra, rb = ring.LocalRing(plan, d), ring.LocalRing(plan, d)
    assert plan.ring_tiles(d) == -(-p // 8192)
    rows = c + N + 1
    ys = ring.y_slots(plan)
    for rep in range(3):
        g = inputs.gradients_numpy(N, d, "normal", seed=20 + rep)
        grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
        for r in (ra, rb):
            r.encode(grads, s)
        for k in range(1, plan.L + 1):
            ra.round(k, s)
        rb.rounds_fused(s)
        torch.cuda.synchronize()
        plan.device_status(s)
        for i in range(N):
            a = ra.ws[i].view(rows, p)[ys]
            b = rb.ws[i].view(rows, p)[ys]
            assert torch.equal(a, b), (rep, i)
    # and the whole aggregation through the fused form against the oracle
    ora = run_oracle(des.U, des.R, g, 0.5)
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    rb.allreduce(grads, outs, 0.5, s, fused=True)
    torch.cuda.synchronize()
    plan.device_status(s)
    assert max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N)) < 5e-6


def test_fused_rounds_give_up_when_a_neighbour_never_answers(mods):
    """One worker's kernel alone: nobody moves its counters, so ring round k = 2 cannot start.  The
    waits run out after the (shortened) limit, the status word says so, nothing hangs and
    the device keeps working."""
    import time
    import torch
    cerar, inputs, ring = mods
    N, c, p = 4, 8, 8192 * 4
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(1))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    s = torch.cuda.current_stream().cuda_stream
    n = plan.rank_workspace_bytes(d) // 4
    ws, peer = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    nt = plan.ring_tiles(d)
    mine, nxt, prv = (torch.zeros(2 * nt, dtype=torch.int32, device="cuda") for _ in range(3))
    assert cerar.cerar_set_tuning("ring_wait_ms", 50) == 0
    try:
        t0 = time.time()
        plan.rank_rounds_fused(1, ws, peer, mine, mine[nt:], nxt, prv[nt:], d, 0, s)
        with pytest.raises(cerar.CerarError) as e:
            plan.device_status(s)
        assert e.value.status == 8                      # CERAR_ERR_TIMEOUT
        assert time.time() - t0 < 10.0
    finally:
        cerar.cerar_set_tuning("ring_wait_ms", 0)
    assert int(nxt[:nt].min()) == 1 and int(prv[nt:].min()) == 1      # ring round k = 1 was done and published
    plan.device_status(s)
    r = ring.LocalRing(plan, d)
    g = inputs.gradients_numpy(N, d, "normal", seed=1)
    grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    r.allreduce(grads, outs, 1.0, s, fused=True)
    torch.cuda.synchronize()
    plan.device_status(s)
    ora = run_oracle(des.U, des.R, g, 1.0)
    assert max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N)) < 5e-6


def test_randomised_ring_shapes(mods):
    """Seeded random (N, c, p): the rank-level path, round by round and with the fused rounds
    (tile size forced small for some, so that short jobs have several tiles), against the oracle."""
    import torch
    cerar, inputs, ring = mods
    rng = np.random.default_rng(31)
    s = torch.cuda.current_stream().cuda_stream
    try:
        for trial in range(16):
            N = int(rng.integers(2, 13))
            c = max(N, int(rng.choice([N, N + 2, 2 * N, 16, 32, 48, 64])))
            p = int(rng.choice([1, 4, 131, 516, 2052, 4104, 9000]))
            tile = int(rng.choice([0, 64, 256, 1024]))
            cerar.cerar_set_tuning("ring_tile", tile)
            d = c * p
            des = Dz.custom_orthogonal(N, c, np.random.default_rng(trial))
            g = inputs.gradients_numpy(N, d, "normal", seed=200 + trial)
            plan = cerar.Plan.create_custom(N, c, des.U, des.R)
            scale = float(rng.choice([1.0, 1.0 / N]))
            ora = run_oracle(des.U, des.R, g, scale)
            r = ring.LocalRing(plan, d)
            grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
            outs = [torch.empty(d, device="cuda") for _ in range(N)]
            for fused in (False, True, True):
                r.allreduce(grads, outs, scale, s, fused=fused)
                torch.cuda.synchronize()
                plan.device_status(s)
                worst = max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N))
                assert worst < 1e-5, (N, c, p, tile, fused, worst)
    finally:
        cerar.cerar_set_tuning("ring_tile", 0)


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 + 260), (3, 5, 1031), (2, 2, 4), (8, 32, 4100), (5, 7, 3)])
def test_round_into_a_message_buffer_equals_the_peer_store(mods, N, c, p):
    """cerar_rank_round_msg forms the same message as cerar_rank_round, bit for bit, but leaves
    it in the caller's buffer; moving the buffers by hand into the neighbours' landing slots (what a
    send / receive pair does) gives the same workspaces, and an unaligned buffer takes the
    scalar path with the same bits."""
    import torch
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(3 * N + c))
    g = inputs.gradients_numpy(N, d, "normal", seed=9)
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    s = torch.cuda.current_stream().cuda_stream
    a, b = ring.LocalRing(plan, d), ring.LocalRing(plan, d)
    grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
    for r in (a, b):
        for w in r.ws:
            w.fill_(float("nan"))
        r.encode(grads, s)
    rows = c + N + 1
    raw = torch.full((N, p + 1), float("nan"), device="cuda")
    for k, _prev, _cancel, _add, land in ring.round_schedule(plan):
        a.round(k, s)
        off = k % 2                                       # odd rounds: a buffer that is not 16-byte aligned
        for i in range(N):
            plan.rank_round_msg(i, b.ws[i], raw[i, off:off + p], d, k, s)
        for i in range(N):                                # every message formed before any lands
            b.ws[(i + 1) % N].view(rows, p)[land].copy_(raw[i, off:off + p])
        for i in range(N):
            assert torch.equal(a.ws[i].view(rows, p)[land], b.ws[i].view(rows, p)[land]), (k, i)
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    b.decode(outs, 1.0 / N, s)
    torch.cuda.synchronize()
    plan.device_status(s)
    ora = run_oracle(des.U, des.R, g, 1.0 / N)
    assert max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N)) < 5e-6
    with pytest.raises(cerar.CerarError):
        plan.rank_round_msg(0, b.ws[0], raw[0, :p], d, 0, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_round_msg(N, b.ws[0], raw[0, :p], d, 1, s)


def _bf16_rounds_on_device(plan, ring_mod, r, d, p, N, s, torch):
    """All L rounds with bfloat16 messages: every worker's message into a 2-byte buffer, then
    "transport" = the neighbour expands that buffer into its landing slot."""
    raw = torch.zeros((N, p + 5), dtype=torch.bfloat16, device="cuda")
    for k in range(1, plan.L + 1):
        off = 1 if k % 3 == 0 else 0                      # every third round: a buffer that is only 2-byte aligned
        for i in range(N):
            plan.rank_round_msg_bf16(i, r.ws[i], raw[i, off:off + p], d, k, s)
        for i in range(N):
            plan.rank_recv_bf16((i + 1) % N, r.ws[(i + 1) % N], raw[i, off:off + p], d, k, s)
    return raw


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 + 260), (3, 5, 1031), (2, 2, 4), (8, 32, 4100), (5, 7, 3), (4, 4, 4096)])
def test_bf16_messages_equal_the_oracle_bit_for_bit(mods, N, c, p):
    """Messages rounded to bfloat16 by the sender (cerar_rank_round_msg_bf16) and expanded by the receiver
    (cerar_rank_recv_bf16).  A rounding is a decision, so both sides take it in binary32 on the SAME encoded
    vectors: seeded synthetic binary32 deltas are written into the D rows of the workspaces (no encode on
    either side) and given to the oracle; the observations Y must then agree bit for bit.  The decode of those
    observations is compared within the usual tolerance."""
    import torch
    from oracle import mixed as Mx
    from oracle import protocol as P
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(5 * N + c))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    s = torch.cuda.current_stream().cuda_stream
    r = ring.LocalRing(plan, d)
    rows = c + N + 1
    delta = inputs.gradients_numpy(N, d, "normal", seed=12)             # worker i's c x p deltas, row-major
    for i in range(N):
        r.ws[i].fill_(float("nan"))
        r.ws[i].view(rows, p)[N + 1:N + 1 + c].copy_(torch.from_numpy(delta[i]).view(c, p))
    _bf16_rounds_on_device(plan, ring, r, d, p, N, s, torch)
    torch.cuda.synchronize()
    plan.device_status(s)
    ys = ring.y_slots(plan)
    Y_dev = [r.ws[i].view(rows, p)[ys].cpu().numpy().T for i in range(N)]                             # p x (L+1)
    Y_ora = Mx.run_rounds_bf16([delta[i].reshape(c, p).T.copy() for i in range(N)])
    for i in range(N):
        assert np.array_equal(Y_dev[i].view(np.uint32), Y_ora[i].view(np.uint32)), i
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    r.decode(outs, 1.0 / N, s)
    torch.cuda.synchronize()
    for i in range(N):
        want = P.unchunk(P.decode(Y_ora[i].astype(np.float64), des.R[i], 1.0 / N))
        assert rel_l2(outs[i].cpu().numpy(), want) < 5e-6
    raw = torch.zeros(p, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cerar.CerarError):
        plan.rank_round_msg_bf16(0, r.ws[0], raw, d, plan.L + 1, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_recv_bf16(N, r.ws[0], raw, d, 1, s)


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 + 260), (8, 32, 4100), (4, 4, 4096)])
def test_bf16_messages_whole_pipeline_within_the_rounding_noise(mods, N, c, p):
    """Encode on the device, rounds with bfloat16 messages, decode, against the oracle's pipeline (fp64
    encode, deltas cast to binary32, rounds of oracle.mixed, fp64 decode).  The two encodes differ by binary32
    rounding (~1e-7 relative), so a rounding decision differs for about 1e-7 / 2^-8 = 3e-5 of the message
    elements per round, each time by one bfloat16 ulp (2^-7 relative): expected relative L2 distance about
    2^-7 sqrt(3e-5 L) ~ 3e-4 at L = 38; tolerance 2e-3.  The distance to the exact protocol is the price of
    8-bit messages with kappa ~ 1."""
    import torch
    from oracle import mixed as Mx
    from oracle import protocol as P
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(5 * N + c))
    g = inputs.gradients_numpy(N, d, "normal", seed=13)
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    s = torch.cuda.current_stream().cuda_stream
    r = ring.LocalRing(plan, d)
    r.encode([torch.from_numpy(g[i]).cuda() for i in range(N)], s)
    _bf16_rounds_on_device(plan, ring, r, d, p, N, s, torch)
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    r.decode(outs, 1.0 / N, s)
    torch.cuda.synchronize()
    plan.device_status(s)
    Delta = [P.encode(P.chunk_matrix(g[i], c), des.U[i]).astype(np.float32) for i in range(N)]
    Y = Mx.run_rounds_bf16(Delta)
    exact = run_oracle(des.U, des.R, g, 1.0 / N)
    worst, worst_exact = 0.0, 0.0
    for i in range(N):
        want = P.unchunk(P.decode(Y[i].astype(np.float64), des.R[i], 1.0 / N))
        worst = max(worst, rel_l2(outs[i].cpu().numpy(), want))
        worst_exact = max(worst_exact, rel_l2(outs[i].cpu().numpy(), exact["out"][i]))
    assert worst < 2e-3, worst
    assert 1e-4 < worst_exact < 2.0 ** -8 * (c + N), worst_exact


def _fp8_rounds_on_device(plan, r, d, N, s, torch, keep_round=None):
    """All L rounds with 8-bit messages: every worker's message (codes + tile scales) into a byte buffer,
    then the neighbour expands that buffer into its landing slot.  Returns the buffers of round keep_round."""
    nbytes = plan.fp8_message_bytes(d)
    raw = torch.full((N, (nbytes + 15) // 16 * 16), 0xAB, dtype=torch.uint8, device="cuda")
    kept = None
    for k in range(1, plan.L + 1):
        for i in range(N):
            plan.rank_round_msg_fp8(i, r.ws[i], raw[i], d, k, s)
        if k == keep_round:
            torch.cuda.synchronize()
            kept = raw.cpu().numpy().copy()
        for i in range(N):
            plan.rank_recv_fp8((i + 1) % N, r.ws[(i + 1) % N], raw[i], d, k, s)
    return kept


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 + 260), (3, 5, 1031), (2, 2, 4), (8, 32, 4100), (5, 7, 3), (4, 4, 4096),
                                   (4, 4, 1024), (3, 6, 2049)])
def test_fp8_messages_equal_the_oracle_bit_for_bit(mods, N, c, p):
    """8-bit messages (cerar_rank_round_msg_fp8 / cerar_rank_recv_fp8): a power-of-two scale per tile of 1024
    positions and an e4m3 code per position.  As for bfloat16, both sides quantise the SAME binary32 encoded
    vectors (seeded synthetic deltas of widely different magnitudes per row, a zero tile included), so
    codes, scales and the observations Y must agree with the oracle bit for bit; ragged last tiles, p not a
    multiple of 4 and p smaller than a tile are among the shapes."""
    import torch
    from oracle import mixed as Mx
    from oracle import protocol as P
    cerar, inputs, ring = mods
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(5 * N + c))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    assert plan.fp8_message_bytes(d) == (p + 15) // 16 * 16 + 4 * ((p + 1023) // 1024)
    s = torch.cuda.current_stream().cuda_stream
    r = ring.LocalRing(plan, d)
    rows = c + N + 1
    delta = inputs.gradients_numpy(N, d, "normal", seed=14).reshape(N, c, p)
    mags = 10.0 ** np.random.default_rng(3).uniform(-6, 6, (N, c, 1))
    delta = (delta * mags).astype(np.float32)
    delta[0, 0, :min(p, 1024)] = 0.0                                       # a tile of zeros in the first message
    for i in range(N):
        r.ws[i].fill_(float("nan"))
        r.ws[i].view(rows, p)[N + 1:N + 1 + c].copy_(torch.from_numpy(delta[i]))
    kept = _fp8_rounds_on_device(plan, r, d, N, s, torch, keep_round=1)
    torch.cuda.synchronize()
    plan.device_status(s)
    # round 1: x_{i,1} = delta_{i,1}; what went on the wire, byte for byte
    off = (p + 15) // 16 * 16
    nt = (p + 1023) // 1024
    for i in range(N):
        codes, scales, _ = Mx.quantize_fp8_tiles(delta[i, 0])
        assert np.array_equal(kept[i, :p], codes), i
        assert np.array_equal(kept[i, off:off + 4 * nt].view(np.float32), scales), i
    ys = ring.y_slots(plan)
    Y_dev = [r.ws[i].view(rows, p)[ys].cpu().numpy().T for i in range(N)]
    Y_ora = Mx.run_rounds_fp8([delta[i].T.copy() for i in range(N)])
    for i in range(N):
        assert np.array_equal(Y_dev[i].view(np.uint32), Y_ora[i].view(np.uint32)), i
    outs = [torch.empty(d, device="cuda") for _ in range(N)]
    r.decode(outs, 1.0 / N, s)
    torch.cuda.synchronize()
    for i in range(N):
        want = P.unchunk(P.decode(Y_ora[i].astype(np.float64), des.R[i], 1.0 / N))
        assert rel_l2(outs[i].cpu().numpy(), want) < 5e-6
    raw = torch.zeros(plan.fp8_message_bytes(d) + 16, dtype=torch.uint8, device="cuda")
    with pytest.raises(cerar.CerarError):
        plan.rank_round_msg_fp8(0, r.ws[0], raw, d, plan.L + 1, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_recv_fp8(N, r.ws[0], raw, d, 1, s)
    with pytest.raises(cerar.CerarError):
        plan.rank_round_msg_fp8(0, r.ws[0], raw.data_ptr() + 4, d, 1, s)          # not 16-byte aligned


def test_message_precision_against_the_condition_number(mods):
    """What low-precision messages cost, by design: decoded relative error (against the fp64 oracle with
    exact messages) for binary32 / bfloat16 / 8-bit messages on a well-conditioned design (c = N) and on one
    with kappa ~ 1e4.  The error follows kappa_2(M_i) times the message precision: usable at c = N, useless
    where kappa times 2^-4 exceeds one."""
    import torch
    from oracle import protocol as P
    cerar, inputs, ring = mods
    p = 4096
    table = []
    for N, c, eps in ((4, 4, 1e-3), (8, 8, 1e-3), (4, 8, 1e-2)):
        d = c * p
        B = inputs.base_matrix(N, c, 0)
        des = Dz.epsilon(N, c, eps, B)
        kap = max(P.kappa2(P.m_matrix(des.U, i)) for i in range(N))
        plan = cerar.Plan.create_custom(N, c, des.U, des.R)
        g = inputs.gradients_numpy(N, d, "normal", seed=15)
        ora = run_oracle(des.U, des.R, g, 1.0 / N)
        s = torch.cuda.current_stream().cuda_stream
        errs = {}
        for kind in ("f32", "bf16", "fp8"):
            r = ring.LocalRing(plan, d)
            r.encode([torch.from_numpy(g[i]).cuda() for i in range(N)], s)
            if kind == "f32":
                for k in range(1, plan.L + 1):
                    r.round(k, s)
            elif kind == "bf16":
                _bf16_rounds_on_device(plan, ring, r, d, p, N, s, torch)
            else:
                _fp8_rounds_on_device(plan, r, d, N, s, torch)
            outs = [torch.empty(d, device="cuda") for _ in range(N)]
            r.decode(outs, 1.0 / N, s)
            torch.cuda.synchronize()
            plan.device_status(s)
            errs[kind] = max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N))
        table.append((N, c, kap, errs))
        print(f"\n[N={N} c={c} kappa_M={kap:.2e}] rel. error of the decoded mean: f32 {errs['f32']:.2e}  "
              f"bf16 {errs['bf16']:.2e}  fp8 {errs['fp8']:.2e}")
        assert errs["f32"] < 4 * kap * 2.0 ** -24 + 1e-6
        assert errs["f32"] < errs["bf16"] < errs["fp8"]
        assert errs["bf16"] < kap * 2.0 ** -8 * 4 and errs["fp8"] < kap * 2.0 ** -4 * 4
    assert table[0][3]["fp8"] < 0.5                                        # c = N: coarse but a mean
    assert table[2][3]["fp8"] > 1.0                                        # kappa ~ 1e4: no correct digit left


def test_rank_level_kernels_on_symmetric_memory_allocations(mods):
    """DistributedRing keeps workspaces and counters in torch's symmetric memory.  With one GPU
    the peer mapping cannot be exercised, but the allocations can: a one-rank NCCL group,
    every worker's workspace and the counters from symm_mem.empty + rendezvous (as the driver
    does, buffers taken through the handle), then the rank-level kernels and the fused rounds
    on them, against the oracle."""
    import os
    import torch
    import torch.distributed as dist
    cerar, inputs, ring = mods
    try:
        import torch.distributed._symmetric_memory as symm_mem
    except Exception as e:                                    # pragma: no cover
        pytest.skip(f"no symmetric memory in this torch: {e}")
    import socket
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if "MASTER_PORT" not in os.environ:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            os.environ["MASTER_PORT"] = str(sk.getsockname()[1])
    created = not dist.is_initialized()
    try:
        if created:
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
        probe = symm_mem.empty(16, dtype=torch.float32, device=torch.device("cuda", 0))
        symm_mem.rendezvous(probe, dist.group.WORLD)
    except Exception as e:                                    # the environment, not the library under test
        if created and dist.is_initialized():
            dist.destroy_process_group()
        pytest.skip(f"symmetric memory cannot be set up here: {e}")
    try:
        N, c, p = 4, 8, 8192 * 2 + 516
        d = c * p
        des = Dz.custom_orthogonal(N, c, np.random.default_rng(8))
        plan = cerar.Plan.create_custom(N, c, des.U, des.R)
        g = inputs.gradients_numpy(N, d, "normal", seed=9)
        ora = run_oracle(des.U, des.R, g, 1.0)
        s = torch.cuda.current_stream().cuda_stream
        n, nt = plan.rank_workspace_bytes(d) // 4, plan.ring_tiles(d)
        dev = torch.device("cuda", 0)
        r = ring.LocalRing(plan, d)
        keep = []
        for i in range(N):
            t = symm_mem.empty(n, dtype=torch.float32, device=dev)
            h = symm_mem.rendezvous(t, dist.group.WORLD)
            r.ws[i] = h.get_buffer(0, (n,), torch.float32)
            keep.append((t, h))
        cnt = symm_mem.empty(2 * N * nt, dtype=torch.int32, device=dev)
        cnt.zero_()
        hc = symm_mem.rendezvous(cnt, dist.group.WORLD)
        r.counters = hc.get_buffer(0, (2 * N * nt,), torch.int32)
        grads = [torch.from_numpy(g[i]).cuda() for i in range(N)]
        outs = [torch.empty(d, device="cuda") for _ in range(N)]
        for fused in (False, True, True):
            r.allreduce(grads, outs, 1.0, s, fused=fused)
            keep[0][1].barrier(channel=0, timeout_ms=5000)     # the driver's stream barrier, one rank
            torch.cuda.synchronize()
            plan.device_status(s)
            assert max(rel_l2(outs[i].cpu().numpy(), ora["out"][i]) for i in range(N)) < 5e-6
    finally:
        if created:
            dist.destroy_process_group()
