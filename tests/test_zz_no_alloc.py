"""cerar_allreduce_sim_static: the pipeline for callers that cannot hand the
library a workspace because they cannot allocate device memory when they call
it (their framework's pool owns all free memory, or an allocation's device-wide
synchronisation is not acceptable inside their step loop).  The workspace is a
fixed 64 MiB array inside the library.

Collected last on purpose (file name), so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.  The test
does not depend on what ran before: it passes alone in a fresh process too.
"""
import numpy as np
import pytest

from oracle import designs as Dz
from tests._harness import rel_l2

pytestmark = pytest.mark.gpu

STATIC_WS_BYTES = 64 * 1024 * 1024


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192 + 260),       # FMA contraction, several tiles and a ragged tail
                                   (8, 32, 4096 + 128)])     # tensor-core contraction: TMA maps on the built-in array
def test_static_workspace_entry_point_matches_the_ordinary_one(N, c, p):
    import torch
    from oracle import protocol as P
    from paper_2609_23898_b200 import cerar, inputs

    assert torch.cuda.is_available()
    d = c * p
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(11))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    assert plan.workspace_bytes(d) <= STATIC_WS_BYTES
    s = torch.cuda.current_stream().cuda_stream
    ws = torch.empty(plan.workspace_bytes(d) // 4, dtype=torch.float32, device="cuda")
    # two calls in a row with different gradients: the second one finds the
    # array full of the first call's values and must not be disturbed by them
    for call, seed in enumerate((21, 22)):
        g_np = inputs.gradients_numpy(N, d, "normal", seed=seed)
        g = torch.from_numpy(g_np).cuda()
        want = torch.full((N, d), float("nan"), dtype=torch.float32, device="cuda")
        got = torch.full((N, d), float("nan"), dtype=torch.float32, device="cuda")
        plan.allreduce_sim(g, d, want, d, ws, d, 1.0 / N, s)                 # existing entry point
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        n0 = plan.launch_count()
        plan.allreduce_sim_static(g, d, got, d, d, 1.0 / N, s)              # new one, no workspace argument
        torch.cuda.synchronize()
        if call == 1:
            # the promise in the name: not a byte of device memory was taken by the call (the first
            # call on a device may be the one that makes the runtime load the array, hence the second)
            assert torch.cuda.mem_get_info()[0] == free_before
        assert plan.launch_count() - n0 == 3                               # encode, rounds, decode ran on the GPU
        plan.device_status(s)
        want_np, got_np = want.cpu().numpy(), got.cpu().numpy()
        assert np.isfinite(got_np).all()
        assert np.array_equal(got_np, want_np), call        # same kernels, same inputs, same order: same bits
        if call == 0:
            # and once against the oracle, so that the test stands by itself
            ora = P.allreduce([x.astype(np.float64) for x in g_np], des.U, des.R, 1.0 / N)
            for i in range(N):
                assert rel_l2(got_np[i], ora["out"][i]) < 5e-6, i
        cnt = plan.counters()
        assert cnt["rounds_done"] == plan.L
        assert cnt["bytes_forwarded_per_worker"] * c == cnt["bytes_gradient"] * (c + N - 2)


def test_static_workspace_checks_the_plan_before_it_touches_the_device():
    """A plan without device copies is refused before the built-in array is looked up (the lookup is what
    loads the array onto the current device)."""
    import torch
    from paper_2609_23898_b200 import cerar

    N, c = 4, 8
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(13))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True)
    g = torch.zeros(N * c * 8, dtype=torch.float32, device="cuda")
    out = torch.zeros(N * c * 8, dtype=torch.float32, device="cuda")
    with pytest.raises(cerar.CerarError) as e:
        plan.allreduce_sim_static(g, c * 8, out, c * 8, c * 8, 1.0)
    assert e.value.status == 6


def test_static_workspace_rejects_what_does_not_fit():
    import torch
    from paper_2609_23898_b200 import cerar

    N, c = 4, 8
    des = Dz.custom_orthogonal(N, c, np.random.default_rng(12))
    plan = cerar.Plan.create_custom(N, c, des.U, des.R)
    p = STATIC_WS_BYTES // (4 * N * (c + N)) + 4                            # one step beyond the capacity
    d = c * p
    assert plan.workspace_bytes(d) > STATIC_WS_BYTES
    g = torch.zeros(N * d, dtype=torch.float32, device="cuda")
    out = torch.zeros(N * d, dtype=torch.float32, device="cuda")
    with pytest.raises(cerar.CerarError) as e:
        plan.allreduce_sim_static(g, d, out, d, d, 1.0)
    assert e.value.status == 9
    assert "64" in str(e.value) or "67108864" in str(e.value)
    with pytest.raises(cerar.CerarError) as e:
        plan.allreduce_sim_static(g, d, out, d, c * 8 + 1, 1.0)              # c does not divide d
    assert e.value.status == 2
