"""cerar_allreduce_fused: the whole protocol in one launch with the slots of all workers
in shared memory.  Same arithmetic as the FMA kernels of the in-HBM pipeline, so besides
matching the oracle it must reproduce that pipeline bit for bit."""
import numpy as np
import pytest

from oracle import designs as Dz
from oracle import protocol as P
from tests._harness import rel_l2, run_oracle

pytestmark = pytest.mark.gpu


def _run_fused(plan, g, scale):
    import torch
    N, d = g.shape
    dev_g = torch.from_numpy(g).cuda()
    out = torch.full((N, d), float("nan"), dtype=torch.float32, device="cuda")
    plan.allreduce_fused(dev_g, d, out, d, d, scale, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192), (4, 8, 8192 + 261), (4, 16, 4097), (8, 8, 1000), (2, 4, 1), (3, 5, 77),
                                   (4, 6, 130), (8, 12, 2050), (4, 32, 515), (8, 16, 384), (4, 4, 100000), (4, 20, 300),
                                   (16, 16, 200)])
def test_fused_matches_oracle_and_the_hbm_pipeline(N, c, p):
    import torch
    from paper_2609_23898_b200 import cerar, inputs
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(100 * N + c))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    if not plan.fused_supported():
        pytest.skip("state does not fit in shared memory")
    d = c * p
    g = inputs.gradients_numpy(N, d, "normal", seed=13)
    scale = 1.0 / N
    got = _run_fused(plan, g, scale)
    ora = run_oracle(des.U, des.R, g, scale)
    assert np.isfinite(got).all()
    assert max(rel_l2(got[i], ora["out"][i]) for i in range(N)) < 5e-6
    cnt = plan.counters()
    assert cnt["rounds_done"] == plan.L
    assert cnt["bytes_forwarded_per_worker"] * c == cnt["bytes_gradient"] * (c + N - 2)
    # bit-identical to the FMA kernels of the in-HBM pipeline (plain kernel: same order of operations)
    plan.set_kernel_mode(cerar.KERNEL_REF)
    dev_g = torch.from_numpy(g).cuda()
    ref = torch.empty(N, d, dtype=torch.float32, device="cuda")
    ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device="cuda")
    plan.allreduce_sim(dev_g, d, ref, d, ws, d, scale, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(got, ref.cpu().numpy())


def test_fused_with_a_paper_design_and_unsupported_shapes():
    from paper_2609_23898_b200 import cerar, inputs
    N, c, p, eps = 4, 8, 4096 + 2, 1e-2
    B = inputs.base_matrix(N, c, 0)
    des = Dz.epsilon(N, c, eps, B)
    plan = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=B)
    g = inputs.gradients_numpy(N, c * p, "normal", seed=14)
    got = _run_fused(plan, g, 1.0)
    ora = run_oracle(des.U, des.R, g, 1.0)
    kap = max(P.kappa2(P.m_matrix(des.U, i)) for i in range(N))
    assert max(rel_l2(got[i], ora["out"][i]) for i in range(N)) < 4 * kap * 2.0 ** -24
    big = Dz.custom_orthogonal(8, 64, np.random.default_rng(0))
    plan_big = cerar.Plan.create_custom(8, 64, big.U, big.R)
    assert not plan_big.fused_supported()
    with pytest.raises(cerar.CerarError) as e:
        _run_fused(plan_big, inputs.gradients_numpy(8, 64 * 16, "normal", seed=1), 1.0)
    assert e.value.status == 1
