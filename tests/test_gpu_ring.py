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
    if c < 32:
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
