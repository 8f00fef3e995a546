"""Host-side logic of the library, no GPU needed: the fp64 plan builder against
the oracle's designs, the exported symbols, argument checking."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import designs as Dz
from oracle import protocol as P
from paper_2609_23898_b200 import cerar, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _plan_mats(pl):
    return [pl.get_U(i) for i in range(pl.N)], [pl.get_R(i) for i in range(pl.N)]


def _normwise(a, b):
    return np.abs(np.asarray(a) - np.asarray(b)).max() / max(np.abs(np.asarray(b)).max(), 1e-300)


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "cerar.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(cerar_[a-z_A-Z0-9]+)\s*\(", header))
    assert {"cerar_plan_create", "cerar_encode", "cerar_ring_round", "cerar_decode",
            "cerar_allreduce_sim", "cerar_get_counters"} <= names
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2609_23898_b200", "libcerar.so"))
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} is declared in cerar.h but not exported"


@pytest.mark.parametrize("N,c,tau", [(4, 8, 0.1), (3, 5, 0.2), (4, 16, 0.05), (2, 2, 0.3), (8, 12, 0.1)])
def test_vandermonde_plan_matches_oracle(N, c, tau):
    pl = cerar.Plan.create(N, c, cerar.VANDERMONDE, tau, host_only=True)
    des = Dz.vandermonde(N, c, tau)
    U, R = _plan_mats(pl)
    for i in range(N):
        assert _normwise(U[i], des.U[i]) < 1e-13
        assert _normwise(R[i], des.R[i]) < 1e-14
    info = pl.info()
    assert info["phi"] == pytest.approx(float(Dz.phi_mp(des)), rel=1e-10)
    assert (info["N"], info["c"], info["L"]) == (N, c, c + N - 2)


@pytest.mark.parametrize("N,c,eps", [(4, 5, 1e-2), (4, 16, 1e-3), (8, 32, 1e-2), (4, 4, 1e-3), (3, 7, 1e-1),
                                     (4, 32, 1e-3), (4, 4, 0.0), (16, 16, 1e-3)])
def test_epsilon_plan_matches_oracle(N, c, eps):
    B = inputs.base_matrix(N, c, 0)
    pl = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=B, host_only=True)
    des = Dz.epsilon(N, c, eps, B)
    U, R = _plan_mats(pl)
    for i in range(N):
        assert _normwise(U[i], des.U[i]) < 1e-12, (i, _normwise(U[i], des.U[i]))
        assert _normwise(R[i], des.R[i]) < 1e-14
    assert pl.info()["phi"] == pytest.approx(float(Dz.phi_mp(des)), rel=1e-10, abs=1e-30)


def test_epsilon_plan_with_custom_h_and_default_B():
    N, c, eps = 3, 6, 5e-2
    h = np.linspace(0.9, -0.7, c)
    B = inputs.base_matrix(N, c, 3)
    pl = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=B, h=h, host_only=True)
    des = Dz.epsilon(N, c, eps, B, list(h))
    for i in range(N):
        assert _normwise(pl.get_U(i), des.U[i]) < 1e-12
    # built-in B: identities that hold for any B (Prop. 1 in block form)
    pl2 = cerar.Plan.create(N, c, cerar.EPSILON, eps, seed=7, host_only=True)
    U, R = _plan_mats(pl2)
    Dinv = np.diag(1.0 / (1.0 + eps * np.array(Dz.default_h(c))))
    for i in range(N):
        for s in range(N):
            blk = U[(i - 1 - s) % N] @ R[i][s:s + c, :]
            np.testing.assert_allclose(blk, np.eye(c) if s >= i else Dinv, atol=1e-8)
    # different seeds give different B, same seed the same
    a = cerar.Plan.create(N, c, cerar.EPSILON, eps, seed=7, host_only=True).get_R(0)
    b = cerar.Plan.create(N, c, cerar.EPSILON, eps, seed=8, host_only=True).get_R(0)
    np.testing.assert_array_equal(a, R[0])
    assert np.abs(a - b).max() > 1e-3
    # the built-in draws look like N(0,1)
    big = cerar.Plan.create(16, 128, cerar.EPSILON, 1e-3, seed=1, host_only=True).get_R(0)[:16, :]
    assert abs(big.mean()) < 0.1 and abs(big.std() - 1.0) < 0.1


def test_kappa_plan_matches_oracle_and_invariants():
    N, c, C = 4, 12, 1e4
    B = inputs.base_matrix(N, c, 0)
    pl = cerar.Plan.create(N, c, cerar.KAPPA, C, B=B, als_iters=40, host_only=True)
    des = Dz.kappa_constrained(N, c, C, B, iters=40)
    U, R = _plan_mats(pl)
    info = pl.info()
    assert info["als_iters_done"] == des.info["iters_done"]
    assert info["phi"] == pytest.approx(P.phi(des.U, des.R), rel=1e-6)
    assert P.phi(U, R) == pytest.approx(info["phi"], rel=1e-8)
    for i in range(N):
        assert _normwise(U[i], des.U[i]) < 1e-6
        assert _normwise(R[i], des.R[i]) < 1e-6
        assert P.kappa2(P.m_matrix(U, i)) <= C
        sv = np.linalg.svd(U[i], compute_uv=False)
        assert sv[0] / sv[-1] <= C / np.sqrt(N) * (1 + 1e-9)
    assert info["kappa_M_max"] == pytest.approx(max(P.kappa2(P.m_matrix(U, i)) for i in range(N)), rel=1e-6)
    assert info["kappa_U_max"] == pytest.approx(max(P.kappa2(u) for u in U), rel=1e-6)


def test_kappa_plan_at_the_fourth_configuration_shape():
    """N = 8, c = 64, C = 1e4 (the fourth configuration).  The initial encoders have kappa ~ 1e15 there,
    so two fp64 implementations of the first projection differ in the small singular directions by about
    1e-4 of ||U_k||, and the least-squares decoder amplifies a change of U by kappa_2(M_i) ~ 4e3: the
    library's and the oracle's U agree to 1e-3, their R only to first order, their Phi to 1e-3.  What
    must hold exactly is checked on the library's own matrices: the projection interval (smallest singular
    value of the initial design, taken from its well-conditioned inverse), the constraint, and that R_i
    is the least-squares decoder of M_i(U) (zero slope of Phi in every R_i)."""
    N, c, C, iters = 8, 64, 1e4, 3
    B = inputs.base_matrix(N, c, 0)
    pl = cerar.Plan.create(N, c, cerar.KAPPA, C, B=B, als_iters=iters, als_tol=1e-300, host_only=True)
    des = Dz.kappa_constrained(N, c, C, B, iters=iters, tol=0.0)
    U, R = _plan_mats(pl)
    info = pl.info()
    assert info["als_iters_done"] == iters
    assert info["phi"] == pytest.approx(P.phi(U, R), rel=1e-8)
    assert info["phi"] == pytest.approx(des.info["phi_history"][-1], rel=1e-3)
    a0, b0 = des.info["a0"], des.info["b0"]
    for i in range(N):
        assert _normwise(U[i], des.U[i]) < 1e-3
        sv = np.linalg.svd(U[i], compute_uv=False)
        assert sv[-1] >= a0 * (1 - 1e-6) and sv[0] <= b0 * (1 + 1e-6)      # the library's interval is the oracle's
        assert sv[0] == pytest.approx(b0, rel=1e-6)                         # and it binds at the top
        M = P.m_matrix(U, i)
        assert P.kappa2(M) <= C
        grad = M.T @ (M @ R[i] - P.target(N, c))
        assert np.abs(grad).max() < 1e-7 * np.abs(M).max() ** 2


def test_custom_plan_roundtrip_and_info():
    rng = np.random.default_rng(0)
    N, c = 3, 5
    des = Dz.custom_orthogonal(N, c, rng)
    pl = cerar.Plan.create_custom(N, c, des.U, des.R, host_only=True)
    for i in range(N):
        np.testing.assert_array_equal(pl.get_U(i), des.U[i])
        np.testing.assert_array_equal(pl.get_R(i), des.R[i])
    info = pl.info()
    assert info["construction"] == 3
    assert info["phi"] == pytest.approx(P.phi(des.U, des.R), rel=1e-10)
    assert info["kappa_U_max"] == pytest.approx(1.0, abs=1e-8)
    assert info["on_device"] == 0


def test_argument_errors():
    for N, c in [(1, 4), (4, 3), (0, 0), (4, 513)]:
        with pytest.raises(cerar.CerarError) as e:
            cerar.Plan.create(N, c, cerar.EPSILON, 1e-2, host_only=True)
        assert e.value.status == 1
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create(4, 8, cerar.VANDERMONDE, -1.0, host_only=True)
    assert e.value.status == 1
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create(4, 8, cerar.EPSILON, 2.0, host_only=True)      # eps ||H|| >= 1
    assert e.value.status == 1
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create(4, 8, cerar.EPSILON, 0.0, host_only=True)      # D = I, c > N: singular windows
    assert e.value.status == 3
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create(4, 8, 9, 0.1, host_only=True)                  # unknown construction
    assert e.value.status == 1
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create(4, 8, cerar.KAPPA, 1.5, host_only=True)        # C <= sqrt(N)
    assert e.value.status == 1
    bad = np.full((2, 2, 2), np.nan)
    with pytest.raises(cerar.CerarError) as e:
        cerar.Plan.create_custom(2, 2, bad, np.zeros((2, 3, 2)), host_only=True)
    assert e.value.status == 3
    # fp32 overflow of the encoders is only checked when uploading; a host-only
    # plan with huge entries is still returned
    pl = cerar.Plan.create(4, 8, cerar.EPSILON, 1e-2, host_only=True)
    assert pl.workspace_bytes(8 * 100) == 4 * 4 * 12 * 100
    assert pl.workspace_bytes(801) == 0
    # data-path calls on a host-only plan fail loudly instead of computing on the CPU
    with pytest.raises(cerar.CerarError) as e:
        pl.encode(0, 800, 0, 800)
    assert e.value.status == 6
    c = pl.counters()
    assert c["rounds_done"] == 0 and c["bytes_forwarded_per_worker"] == 0
    assert cerar.lib.cerar_status_string(5) == b"call out of order"


def test_design_gamma_matches_oracle_and_selects_the_best_h():
    """cerar_design_gamma against the oracle's K^(l) matrices, and the helper that picks H
    among several trial diagonals, on fixed candidates."""
    from oracle import designs as Dz
    from paper_2609_23898_b200 import cerar, inputs
    rng = np.random.default_rng(9)
    for (N, c) in [(4, 4), (4, 10), (3, 7), (8, 32), (5, 9), (4, 16)]:
        B = inputs.base_matrix(N, c, 0)
        cands = [np.array(Dz.default_h(c))] + [rng.uniform(-1, 1, c) for _ in range(4)]
        for h in cands:
            g_lib = cerar.design_gamma(N, c, B, h)
            g_ora = Dz.gamma(B, h, N, c)
            assert g_lib == pytest.approx(g_ora, rel=1e-8, abs=1e-14)
        best, gammas = cerar.select_h(N, c, B, cands)
        assert gammas[best] == max(gammas)
        assert best == int(np.argmax([Dz.gamma(B, h, N, c) for h in cands]))
    # h = NULL means the equally spaced default; B = NULL the built-in generator (seeded)
    B = inputs.base_matrix(4, 10, 0)
    assert cerar.design_gamma(4, 10, B) == pytest.approx(Dz.gamma(B, Dz.default_h(10), 4, 10), rel=1e-8)
    assert cerar.design_gamma(4, 10, seed=1) > 0 and cerar.design_gamma(4, 10, seed=1) != cerar.design_gamma(4, 10, seed=2)
    with pytest.raises(cerar.CerarError):
        cerar.design_gamma(4, 3)


def test_tradeoff_report_runs_on_the_host(capsys, monkeypatch):
    import sys as _sys
    from paper_2609_23898_b200 import tradeoff
    monkeypatch.setattr(_sys, "argv", ["tradeoff", "--N", "3", "--c", "7", "--trials", "3", "--als-iters", "5"])
    tradeoff.main()
    out = capsys.readouterr().out
    assert "gamma(B, H)" in out and out.count("\n|---|") == 2
    rows = [ln for ln in out.splitlines() if ln.startswith("| 0.001 |")]
    assert len(rows) == 1 and "nan" not in rows[0]


def test_library_kappa_design_reaches_phi_zero_when_c_equals_N():
    """The exactly solvable case c = N: the library's ALS must end at Phi ~ 0 within its bound,
    as the oracle's does."""
    from paper_2609_23898_b200 import cerar, inputs
    for N, C in [(3, 1e6), (4, 1e4)]:
        B = inputs.base_matrix(N, N, 0)
        p = cerar.Plan.create(N, N, cerar.KAPPA, C, B=B, als_iters=1000, als_tol=1e-30, host_only=True)
        info = p.info()
        assert info["phi"] < 1e-18 and info["kappa_M_max"] <= C


def test_padded_length():
    from oracle import designs as Dz
    from paper_2609_23898_b200 import cerar
    des = Dz.custom_orthogonal(4, 12, np.random.default_rng(0))
    plan = cerar.Plan.create_custom(4, 12, des.U, des.R, host_only=True)
    assert plan.padded_length(1_414_647_808) == 1_414_647_840 and 1_414_647_840 % 48 == 0
    assert plan.padded_length(48) == 48 and plan.padded_length(49) == 96 and plan.padded_length(1) == 48
    assert plan.padded_length(0) == 0


@pytest.mark.parametrize("N,c", [(3, 5), (4, 8), (2, 6), (4, 12)])
def test_optimize_h_matches_the_oracle_and_feeds_a_plan(N, c):
    """cerar_design_optimize_h against oracle.designs.optimize_h (same start, same grid, same B): the same
    diagonal, the same gamma; and the diagonal goes into a plan whose diagnostics are the oracle's."""
    from oracle import designs as Dz
    from oracle import protocol as P
    from paper_2609_23898_b200 import cerar
    B = np.random.default_rng(30 + N + c).standard_normal((N, c))
    h_o, g_o, m_o = Dz.optimize_h(B, N, c, sweeps=3, grid=9)
    h_l, g_l, m_l = cerar.optimize_h(N, c, B, sweeps=3, grid=9)
    assert m_l == m_o and np.allclose(h_l, h_o, atol=1e-15)
    assert g_l == pytest.approx(g_o, rel=1e-9)
    assert g_l >= cerar.design_gamma(N, c, B) * (1 - 1e-12)
    # a start of the caller's, here the reversed default
    h0 = np.linspace(1.0, -1.0, c)
    h_o2, g_o2, _ = Dz.optimize_h(B, N, c, h0=h0, sweeps=2, grid=9)
    h_l2, g_l2, _ = cerar.optimize_h(N, c, B, h0=h0, sweeps=2, grid=9)
    assert np.allclose(h_l2, h_o2, atol=1e-15) and g_l2 == pytest.approx(g_o2, rel=1e-9)
    plan = cerar.Plan.create(N, c, cerar.EPSILON, 1e-2, B=B, h=h_l, host_only=True)
    des = Dz.epsilon(N, c, 1e-2, B, h=h_o)
    info = plan.info()
    assert info["phi"] == pytest.approx(P.phi(des.U, des.R), rel=1e-6)
    for i in range(N):
        assert np.allclose(plan.get_U(i), des.U[i], rtol=1e-8, atol=1e-8 * np.abs(des.U[i]).max())
    with pytest.raises(cerar.CerarError):
        cerar.optimize_h(N, c, B, h0=np.zeros(c))
    with pytest.raises(cerar.CerarError):
        cerar.optimize_h(N, c, B, grid=2)


@pytest.mark.parametrize("N,c", [(4, 8), (4, 16), (8, 32)])
def test_block_structured_base_matrix_gives_block_sparse_designs(N, c):
    """A base matrix whose rows have disjoint supports (row r on its own c/N columns) makes every window A_l
    block diagonal up to a permutation, hence U_k and the decoder rows block sparse: c/N non-zeros per column
    of U_k instead of c.  Prop. 1 and Prop. 2 hold for any B with invertible windows, so the design is as valid
    as a dense one; the library and the oracle agree on it, zeros included."""
    from oracle import designs as Dz
    from oracle import protocol as P
    from paper_2609_23898_b200 import cerar, inputs
    B, h = inputs.structured_base(N, c, 1)
    beta = c // N
    eps = 1e-2
    plan = cerar.Plan.create(N, c, cerar.EPSILON, eps, B=B, h=h, host_only=True)
    des = Dz.epsilon(N, c, eps, B, h=h)
    D = 1.0 + eps * h
    assert P.phi(des.U, des.R) == pytest.approx(N * (N - 1) / 2 * np.sum((1.0 / D - 1.0) ** 2), rel=1e-6)   # Prop. 2 (phi from fp64 U, R with kappa up to 1e9)
    for i in range(N):
        U, R = plan.get_U(i), plan.get_R(i)
        assert np.array_equal(U != 0, des.U[i] != 0) and np.array_equal(R != 0, des.R[i] != 0)
        assert np.all((U != 0).sum(axis=0) == beta) and np.all((U != 0).sum(axis=1) == beta)
        assert np.all((R != 0).sum(axis=1) == beta)                      # a decoder row is one a_l: one block
        assert np.allclose(U, des.U[i], rtol=1e-9, atol=1e-9 * np.abs(des.U[i]).max())
        assert np.allclose(R, des.R[i], rtol=1e-9, atol=1e-12)
    # the decoded sum is exact up to the O(eps) of every MPC design (worker 0 exactly)
    rng = np.random.default_rng(2)
    g = [rng.standard_normal(c * 3) for _ in range(N)]
    res = P.allreduce(g, des.U, des.R, 1.0)
    assert P.rel_l2(res["out"][0], P.exact_sum(g)) < 1e-6 * max(1.0, P.kappa2(P.m_matrix(des.U, 0)) * 1e-10)
    assert max(P.rel_l2(res["out"][i], P.exact_sum(g)) for i in range(N)) < 0.2

