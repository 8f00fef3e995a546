"""Pins for oracle.designs: identities and scaling laws the paper states."""
import os
from math import ceil

import mpmath as mp
import numpy as np
import pytest

from oracle import designs as Dz
from oracle import protocol as P


def _maxabs(M):
    return max(abs(M[i, j]) for i in range(M.rows) for j in range(M.cols))


def _rng_B(N, c, seed=0):
    return np.random.default_rng(seed).standard_normal((N, c))


# ------------------------------------------------------------------ MPC core

@pytest.mark.parametrize("N,c", [(2, 3), (3, 3), (4, 5), (4, 10), (5, 12)])
def test_prop1_block_identity_diagonal_D(N, c):
    """U_{i-1-s} W_s(R_i) = I (s >= i) or D^{-1} (s < i)."""
    des = Dz.epsilon(N, c, 3e-2, _rng_B(N, c, N + c))
    with mp.workdps(Dz.DEFAULT_DPS):
        Dinv = mp.inverse(des.Dmat_mp)
        for (i, s), blk in Dz.block_products_mp(des).items():
            ref = mp.eye(c) if s >= i else Dinv
            assert _maxabs(blk - ref) < mp.mpf(10) ** (-60)


def test_prop1_and_prop2_full_matrix_D():
    """Same identities with a non-diagonal perturbation H (general path with
    negative powers of D)."""
    N, c, eps = 3, 5, 2e-2
    rng = np.random.default_rng(42)
    B = rng.standard_normal((N, c))
    H = rng.standard_normal((c, c))
    H /= np.linalg.norm(H, 2)
    Dm = np.eye(c) + eps * H
    des = Dz.mpc(B.tolist(), mp.matrix(Dm.tolist()), N, c)
    with mp.workdps(Dz.DEFAULT_DPS):
        Dinv = mp.inverse(des.Dmat_mp)
        for (i, s), blk in Dz.block_products_mp(des).items():
            ref = mp.eye(c) if s >= i else Dinv
            assert _maxabs(blk - ref) < mp.mpf(10) ** (-60)
        E = Dinv - mp.eye(c)
        closed = mp.mpf(N * (N - 1)) / 2 * sum(E[a, b] ** 2 for a in range(c) for b in range(c))
        assert abs(Dz.phi_mp(des) - closed) < mp.mpf(10) ** (-60)


def test_window_shift_identity():
    """A_{l+N} = A_l D."""
    N, c, eps = 4, 6, 1e-2
    B = _rng_B(N, c, 1)
    with mp.workdps(Dz.DEFAULT_DPS):
        Dv = [1 + mp.mpf(eps) * mp.mpf(h) for h in Dz.default_h(c)]
        Bm = mp.matrix(B.tolist())
        for l in (-3, 0, 2, 5):
            A0 = Dz.window_mp(Bm, Dv, N, c, l)
            A1 = Dz.window_mp(Bm, Dv, N, c, l + N)
            assert _maxabs(A1 - A0 * mp.diag(Dv)) < mp.mpf(10) ** (-80)


def test_prop2_closed_form_value():
    """Phi = N(N-1)/2 ||D^{-1} - I||_F^2, including the fp64 evaluation for a
    mild design."""
    N, c, eps = 4, 5, 1e-2
    des = Dz.epsilon(N, c, eps, _rng_B(N, c))
    closed = N * (N - 1) / 2 * sum((1 / (1 + eps * h) - 1) ** 2 for h in Dz.default_h(c))
    assert float(Dz.phi_mp(des)) == pytest.approx(closed, rel=1e-12)
    assert P.phi(des.U, des.R) == pytest.approx(closed, rel=1e-6)


def test_decoder_rows_and_windows():
    """R_i[l,:] = a_{l-i}; W_s(R_i) = A_{s-i}; U_k A_{N-1-k} = I."""
    N, c = 4, 6
    B = _rng_B(N, c, 2)
    des = Dz.epsilon(N, c, 0.05, B)
    with mp.workdps(Dz.DEFAULT_DPS):
        Dv = [1 + mp.mpf(0.05) * mp.mpf(h) for h in Dz.default_h(c)]
        Bm = mp.matrix(B.tolist())
        for i in range(N):
            for s in range(N):
                A = Dz.window_mp(Bm, Dv, N, c, s - i)
                assert _maxabs(des.R_mp[i][s:s + c, :] - A) < mp.mpf(10) ** (-80)
        for k in range(N):
            A = Dz.window_mp(Bm, Dv, N, c, N - 1 - k)
            assert _maxabs(des.U_mp[k] * A - mp.eye(c)) < mp.mpf(10) ** (-60)
    # first rows of the sequence are the rows of B itself
    np.testing.assert_allclose(des.R[0][:N, :], B, rtol=1e-15)


def test_phi_positive_when_c_exceeds_N():
    """Lemma 1: no finite design reaches Phi = 0 for c > N."""
    for (N, c) in [(3, 4), (4, 9)]:
        for eps in (1e-1, 1e-3, 1e-6):
            des = Dz.epsilon(N, c, eps, _rng_B(N, c))
            assert Dz.phi_mp(des) > 0
        assert Dz.phi_mp(Dz.vandermonde(N, c, 1e-3)) > 0


# ------------------------------------------------------------------ Vandermonde

@pytest.mark.parametrize("N,c,tau", [(4, 6, 0.1), (3, 5, 0.02), (4, 8, 0.1)])
def test_vandermonde_phi_closed_form(N, c, tau):
    des = Dz.vandermonde(N, c, tau)
    xi = Dz.default_xi(c)
    closed = N * (N - 1) / 2 * sum((np.exp(-N * tau * x) - 1) ** 2 for x in xi)
    assert float(Dz.phi_mp(des)) == pytest.approx(closed, rel=1e-12)


def test_vandermonde_leading_term_and_limit():
    """Phi = N^3 (N-1)/2 tau^2 sum xi^2 + O(tau^3): the ratio to the leading
    term tends to 1 and Phi -> 0 as tau -> 0."""
    N, c = 4, 6
    xi = Dz.default_xi(c)
    lead = lambda t: N ** 3 * (N - 1) / 2 * t * t * sum(x * x for x in xi)
    prev = None
    for tau in (1e-1, 1e-2, 1e-3):
        ph = float(Dz.phi_mp(Dz.vandermonde(N, c, tau)))
        ratio = ph / lead(tau)
        assert abs(ratio - 1) < 30 * tau
        if prev is not None:
            assert ph < prev / 50
        prev = ph
    # worked value: N=4, c=6, tau=0.1 gives 2.8952 against a leading term 2.688
    assert float(Dz.phi_mp(Dz.vandermonde(4, 6, 0.1))) == pytest.approx(2.8952, abs=5e-4)
    assert lead(0.1) == pytest.approx(2.688, abs=1e-3)


def test_vandermonde_entries_and_conditioning():
    N, c, tau = 3, 5, 0.2
    des = Dz.vandermonde(N, c, tau)
    z = np.exp(tau * np.array(Dz.default_xi(c)))
    # R_0 rows are a_l = [z_j^l], l = 0..L
    for l in range(des.L + 1):
        np.testing.assert_allclose(des.R[0][l], z ** l, rtol=1e-14)
    # R_i rows are a_{l-i}, negative powers included
    np.testing.assert_allclose(des.R[2][0], z ** (-2.0), rtol=1e-14)
    # kappa(U_k) grows without bound as tau decreases (Remark 2)
    ks = [max(P.kappa2(u) for u in Dz.vandermonde(N, c, t).U) for t in (0.4, 0.2, 0.1, 0.05)]
    assert all(b > 5 * a for a, b in zip(ks, ks[1:]))


# ------------------------------------------------------------------ epsilon-construction

def test_epsilon_phi_bound_and_quadratic_scaling():
    N, c = 4, 10
    B = _rng_B(N, c)
    h = np.array(Dz.default_h(c))
    vals = []
    for eps in (1e-1, 1e-2, 1e-3):
        ph = float(Dz.phi_mp(Dz.epsilon(N, c, eps, B)))
        bound = N * (N - 1) / 2 * eps ** 2 * np.sum(h ** 2) / (1 - eps * np.max(np.abs(h))) ** 2
        assert 0 < ph <= bound * (1 + 1e-12)
        vals.append(ph)
    assert vals[0] / vals[1] == pytest.approx(100, rel=0.3)
    assert vals[1] / vals[2] == pytest.approx(100, rel=0.03)


@pytest.mark.parametrize("N,c", [(4, 10), (4, 8), (3, 7)])
def test_singular_value_hierarchy_and_kappa_slope(N, c):
    """Theorem 2 / Corollary 1: the singular values of A_l(eps) fall in groups
    Theta(eps^j) with N members for j < beta and s members at j = beta;
    kappa_2(A_l) = Theta(eps^-r*), r* = ceil(c/N) - 1."""
    beta, s = divmod(c, N)
    rstar = ceil(c / N) - 1
    B = _rng_B(N, c)
    h = Dz.default_h(c)
    kap = {}
    svs = {}
    with mp.workdps(Dz.DEFAULT_DPS):
        Bm = mp.matrix(B.tolist())
        for eps in (1e-3, 1e-4, 1e-5):
            Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h]
            for l in range(N):
                sv = [float(v) for v in Dz.singular_values_mp(Dz.window_mp(Bm, Dv, N, c, l))]
                svs[(eps, l)] = sv
                kap.setdefault(l, []).append(sv[0] / sv[-1])
    expect = sorted([j for j in range(beta) for _ in range(N)] + [beta] * s)
    for l in range(N):
        # exponent of eps carried by the t-th singular value, from one decade of eps
        expo = [np.log10(a / b) for a, b in zip(svs[(1e-4, l)], svs[(1e-5, l)])]
        assert [int(round(e)) for e in expo] == expect, (l, expo)
        assert max(abs(e - round(e)) for e in expo) < 0.1
    for l, ks in kap.items():
        slope1 = np.log10(ks[1] / ks[0])      # per decade of eps
        slope2 = np.log10(ks[2] / ks[1])
        assert slope1 == pytest.approx(rstar, abs=0.15)
        assert slope2 == pytest.approx(rstar, abs=0.05)


def test_worked_kappa_values_n4_c10():
    """kappa_2 of the encoders for N=4, c=10, B from numpy seed 0, H =
    diag(linspace(-1,1)): decades of eps change kappa by 10^r* = 100."""
    N, c = 4, 10
    B = _rng_B(N, c)
    ks = []
    for eps in (1e-1, 1e-2, 1e-3):
        des = Dz.epsilon(N, c, eps, B)
        with mp.workdps(Dz.DEFAULT_DPS):
            k = max(float(sv[0] / sv[-1]) for sv in (Dz.singular_values_mp(u) for u in des.U_mp))
        ks.append(k)
    assert ks[1] / ks[0] == pytest.approx(100, rel=0.25)
    assert ks[2] / ks[1] == pytest.approx(100, rel=0.05)


def test_kappa_M_bound():
    """kappa_2(M_j) <= sqrt(N) max sigma_max(U) / min sigma_min(U), and
    sigma_max(M_j) >= max_k sigma_max(U_k) (appendix on U vs M conditioning)."""
    N, c = 4, 7
    des = Dz.epsilon(N, c, 1e-1, _rng_B(N, c))
    smax = max(np.linalg.svd(u, compute_uv=False)[0] for u in des.U)
    smin = min(np.linalg.svd(u, compute_uv=False)[-1] for u in des.U)
    for j in range(N):
        sv = np.linalg.svd(P.m_matrix(des.U, j), compute_uv=False)
        assert sv[0] / sv[-1] <= np.sqrt(N) * smax / smin * (1 + 1e-9)
        assert sv[0] >= smax * (1 - 1e-9)
        assert sv[-1] >= smin * (1 - 1e-9)


def test_finite_difference_matrix(golden_dir):
    F3 = np.loadtxt(os.path.join(golden_dir, "f3.txt"), comments="#")
    np.testing.assert_array_equal(Dz.finite_difference_matrix(3), F3)
    for n in range(1, 9):
        assert round(np.linalg.det(Dz.finite_difference_matrix(n).astype(float))) == 1


def test_finite_difference_identity():
    """Lemma 2: sum_k (-1)^(j-k) C(j,k) b D^(m+k) = eps^j b D^m H^j, and the
    factorisation F Pi A_l = Lambda K_l on a full window."""
    rng = np.random.default_rng(4)
    c, eps = 6, 1e-2
    H = rng.standard_normal((c, c))
    Dm = np.eye(c) + eps * H
    b = rng.standard_normal(c)
    for m in (0, 1, 2):
        for j in range(4):
            F = Dz.finite_difference_matrix(j + 1)
            lhs = sum(F[j, k] * b @ np.linalg.matrix_power(Dm, m + k) for k in range(j + 1))
            rhs = eps ** j * b @ np.linalg.matrix_power(Dm, m) @ np.linalg.matrix_power(H, j)
            np.testing.assert_allclose(lhs, rhs, atol=1e-12 * max(1, np.abs(lhs).max()))
    # whole window, diagonal H, N=3, c=7 (beta=2, s=1), l=1
    N, c, l, eps = 3, 7, 1, 1e-3
    B = _rng_B(N, c, 8)
    h = Dz.default_h(c)
    with mp.workdps(60):
        Bm = mp.matrix(B.tolist())
        Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h]
        A = Dz.window_mp(Bm, Dv, N, c, l, 60)
        idx = list(range(l, l + c))
        for alpha in range(N):
            rows = [t for t, jj in enumerate(idx) if jj % N == alpha]   # grouped by remainder
            n = len(rows)
            m0 = 0 if alpha >= l else 1
            F = Dz.finite_difference_matrix(n)
            for j in range(n):
                lhs = [sum(int(F[j, k]) * A[rows[k], col] for k in range(j + 1)) for col in range(c)]
                rhs = [mp.mpf(eps) ** j * Bm[alpha, col] * Dv[col] ** m0 * mp.mpf(h[col]) ** j for col in range(c)]
                assert max(abs(a - b) for a, b in zip(lhs, rhs)) < mp.mpf(10) ** (-50)


def test_k_limit_rows_are_the_limit_of_the_factorised_window():
    """K^(l)(B, H) against the factorisation it comes from: F~ Pi A_l(eps) = Lambda K_l(eps)
    (checked above), K_l(eps) -> K^(l) as eps -> 0 up to the order of the rows."""
    for (N, c) in [(3, 7), (4, 10), (4, 8), (5, 5)]:
        B = _rng_B(N, c, 21)
        h = np.array(Dz.default_h(c))
        for l in range(N):
            eps = 1e-9
            with mp.workdps(80):
                Bm = mp.matrix(B.tolist())
                Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h.tolist()]
                A = Dz.window_mp(Bm, Dv, N, c, l, 80)
                idx = list(range(l, l + c))
                rows_eps = []
                for alpha in range(N):
                    rows = [t for t, jj in enumerate(idx) if jj % N == alpha]
                    F = Dz.finite_difference_matrix(len(rows))
                    for j in range(len(rows)):
                        r = [sum(int(F[j, k]) * A[rows[k], col] for k in range(j + 1)) / mp.mpf(eps) ** j
                             for col in range(c)]
                        rows_eps.append(np.array([float(x) for x in r]))
            K = Dz.k_limit(B, h, N, c, l)
            assert K.shape == (c, c)
            # same rows, some order: match each limit row to its nearest row of K
            used = set()
            for r in rows_eps:
                dist = np.abs(K - r).max(axis=1)
                t = int(np.argmin(dist))
                assert dist[t] < 1e-6 and t not in used
                used.add(t)


def test_gamma_special_case_and_lower_bound_on_sigma_min():
    """c = N: K^(l) = B, so gamma = sigma_min(B).  And from A_l = Pi^T F~^-1 Lambda K_l:
    sigma_min(A_l(eps)) >= eps^r* sigma_min(K_l(eps)) / ||F~||_2, with sigma_min(K_l(eps))
    within O(eps) of sigma_min(K^(l)) >= gamma."""
    B = _rng_B(5, 5, 3)
    assert Dz.gamma(B, Dz.default_h(5), 5, 5) == pytest.approx(np.linalg.svd(B, compute_uv=False)[-1], rel=1e-12)
    N, c = 4, 10
    beta, s = divmod(c, N)
    r_star = -(-c // N) - 1
    B = _rng_B(N, c, 5)
    h = Dz.default_h(c)
    g = Dz.gamma(B, h, N, c)
    assert g > 0
    normF = max(np.linalg.norm(Dz.finite_difference_matrix(n).astype(float), 2) for n in (beta, beta + 1))
    for eps in (1e-2, 1e-3):
        for l in range(N):
            with mp.workdps(80):
                Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h]
                A = Dz.window_mp(mp.matrix(B.tolist()), Dv, N, c, l, 80)
                smin = float(Dz.singular_values_mp(A, 80)[-1])
            assert smin >= eps ** r_star * (g - 20 * eps) / normF
            assert smin <= 1e3 * eps ** r_star            # and not a different power of eps


@pytest.mark.parametrize("N,c", [(3, 5), (4, 8), (2, 6)])
def test_optimize_h_is_a_coordinatewise_maximum_of_gamma(N, c):
    """The deterministic H: gamma never decreases, ||H|| stays 1, the result cannot be improved by moving
    any single coordinate to any grid value (brute force), and it is reproducible."""
    B = _rng_B(N, c, 21)
    grid = 9
    h0 = Dz.default_h(c)
    g0 = Dz.gamma(B, np.asarray(h0, float), N, c)
    h, g, moves = Dz.optimize_h(B, N, c, sweeps=6, grid=grid)
    assert g >= g0 and moves >= 1 and g > g0 * 1.01                 # it does find something better than the start
    assert g == pytest.approx(Dz.gamma(B, h, N, c), rel=1e-12)
    assert np.abs(h).max() == 1.0
    cand = [-1.0 + 2.0 * t / (grid - 1) for t in range(grid)]
    assert all(min(abs(x - g_) for g_ in cand) < 1e-15 or x in np.asarray(h0, float) / np.abs(h0).max() for x in h)
    for j in range(c):                                              # no single move helps any more
        for v in cand:
            t = h.copy()
            t[j] = v
            if np.abs(t).max() < 1.0:
                continue
            assert Dz.gamma(B, t, N, c) <= g * (1 + 1e-9), (j, v)
    h2, g2, _ = Dz.optimize_h(B, N, c, sweeps=6, grid=grid)
    assert np.array_equal(h, h2) and g == g2
    # and the design built with it is a valid epsilon-construction with a smaller kappa at the same Phi order
    des0 = Dz.epsilon(N, c, 1e-2, B)
    des1 = Dz.epsilon(N, c, 1e-2, B, h=h)
    k0 = max(P.kappa2(P.m_matrix(des0.U, i)) for i in range(N))
    k1 = max(P.kappa2(P.m_matrix(des1.U, i)) for i in range(N))
    assert P.phi(des1.U, des1.R) < 10 * P.phi(des0.U, des0.R) and k1 < 10 * k0


# ------------------------------------------------------------------ kappa-constrained

def test_kappa_constrained_invariants():
    N, c, C = 4, 12, 1e4
    des = Dz.kappa_constrained(N, c, C, _rng_B(N, c), iters=40)
    a0, b0 = des.info["a0"], des.info["b0"]
    assert np.sqrt(N) * b0 / a0 <= C * (1 + 1e-12)
    for u in des.U:
        sv = np.linalg.svd(u, compute_uv=False)
        assert sv[-1] >= a0 * (1 - 1e-9) and sv[0] <= b0 * (1 + 1e-9)
    for i in range(N):
        assert P.kappa2(P.m_matrix(des.U, i)) <= C
    # least-squares steps never increase Phi (before the projection)
    for before, after_U, _ in des.info["steps"]:
        assert after_U <= before * (1 + 1e-9) + 1e-12
    # R is the least-squares decoder for the final U
    for i in range(N):
        M = P.m_matrix(des.U, i)
        grad = M.T @ (M @ des.R[i] - P.target(N, c))
        assert np.abs(grad).max() < 1e-6 * max(1.0, np.abs(M).max() ** 2)
    ph = P.phi(des.U, des.R)
    assert 0 < ph < 1.0
    # improves on simply clipping the initial design
    assert ph <= des.info["phi_history"][0] * (1 + 1e-9)
    # the error it gives on i.i.d. gradients is a few percent (same order as the
    # paper's training-time figure for N=4, c=12; plausibility only)
    rng = np.random.default_rng(1)
    g = [rng.standard_normal(c * 64) for _ in range(N)]
    res = P.allreduce(g, des.U, des.R)
    err = max(P.rel_l2(res["out"][i], P.exact_sum(g)) for i in range(N))
    assert 1e-3 < err < 0.1


# The three steps of one iteration (Sec. II-D), each against the property that defines it.  Phi is
# evaluated from the M_i matrices (pinned by brute force in test_oracle_protocol.py), so a step that
# solved for the wrong blocks, or transposed its result, is not a minimiser of THIS Phi.

def _phi_slope_and_rise(U, R, perturb, t=1e-3):
    """Phi is quadratic along any line: central difference = exact slope, Phi(+t) + Phi(-t) - 2 Phi(0) = 2 t^2 curvature."""
    f0 = P.phi(U, R)
    fp = P.phi(*perturb(U, R, +t))
    fm = P.phi(*perturb(U, R, -t))
    return (fp - fm) / (2 * t), fp + fm - 2 * f0, f0


@pytest.mark.parametrize("N,c", [(3, 5), (4, 6), (2, 5)])
def test_als_U_step_and_R_step_are_stationary_minimisers_of_phi(N, c):
    rng = np.random.default_rng(N * 10 + c)
    L = c + N - 2
    # U-step: R arbitrary, U = argmin_U Phi(U, R)
    R = [rng.standard_normal((L + 1, c)) for _ in range(N)]
    U = Dz._ls_U(R, N, c)
    for trial in range(12):
        k = trial % N
        E = rng.standard_normal((c, c))

        def perturb(U_, R_, t, k=k, E=E):
            V = [u.copy() for u in U_]
            V[k] = V[k] + t * E
            return V, R_
        slope, rise, f0 = _phi_slope_and_rise(U, R, perturb)
        assert abs(slope) < 1e-7 * max(1.0, f0), (k, slope)
        assert rise > 0
    # and it is not a minimiser by accident of the test: a U that is not the step's has a slope
    V = [u + 0.1 * rng.standard_normal((c, c)) for u in U]
    E = rng.standard_normal((c, c))
    slope, _, f0 = _phi_slope_and_rise(V, R, lambda U_, R_, t: ([U_[0] + t * E] + list(U_[1:]), R_))
    assert abs(slope) > 1e-3
    # R-step: U arbitrary, R = argmin_R Phi(U, R)
    U = [rng.standard_normal((c, c)) for _ in range(N)]
    R = Dz._ls_R(U, N, c)
    for trial in range(12):
        i = trial % N
        E = rng.standard_normal((L + 1, c))

        def perturb(U_, R_, t, i=i, E=E):
            Q = [r.copy() for r in R_]
            Q[i] = Q[i] + t * E
            return U_, Q
        slope, rise, f0 = _phi_slope_and_rise(U, R, perturb)
        assert abs(slope) < 1e-7 * max(1.0, f0), (i, slope)
        assert rise > 0


def test_als_projection_is_the_nearest_matrix_with_singular_values_in_the_interval():
    """Clamping the singular values is the Frobenius-nearest point of {sigma(X) in [a, b]}
    (Mirsky's inequality: ||A - X||_F >= ||sigma(A) - sigma(X)||_2, attained with A's singular vectors).
    Checked against that bound, against feasible competitors, and on matrices it must not change."""
    rng = np.random.default_rng(4)
    c, a, b = 5, 0.5, 2.0
    for trial in range(6):
        A = rng.standard_normal((c, c)) * rng.choice([0.3, 1.0, 3.0])
        Pj = Dz._project([A], a, b)[0]
        sA = np.linalg.svd(A, compute_uv=False)
        sP = np.linalg.svd(Pj, compute_uv=False)
        assert sP[-1] >= a * (1 - 1e-12) and sP[0] <= b * (1 + 1e-12)
        best = np.linalg.norm(sA - np.clip(sA, a, b))
        assert np.linalg.norm(A - Pj) == pytest.approx(best, rel=1e-10, abs=1e-13)
        for _ in range(200):                               # no feasible competitor is nearer
            X, _ = np.linalg.qr(rng.standard_normal((c, c)))
            Z, _ = np.linalg.qr(rng.standard_normal((c, c)))
            mix = rng.uniform(0, 0.2)
            Xc, s0, Zc = np.linalg.svd(A)
            Xn, _ = np.linalg.qr(Xc + mix * X)
            Zn, _ = np.linalg.qr(Zc.T + mix * Z)
            comp = (Xn * rng.uniform(a, b, c)) @ Zn.T
            assert np.linalg.norm(A - comp) >= np.linalg.norm(A - Pj) * (1 - 1e-12)
    inside = (np.linalg.qr(rng.standard_normal((c, c)))[0] * rng.uniform(a, b, c)) @ np.linalg.qr(rng.standard_normal((c, c)))[0]
    assert np.allclose(Dz._project([inside], a, b)[0], inside, atol=1e-13)
    once = Dz._project([A], a, b)
    assert np.allclose(Dz._project(once, a, b)[0], once[0], atol=1e-13)


def _max_slope(U, R, which, rng, N, c, trials=6):
    """Largest |d Phi / dt| over random unit directions in the U_k (which = "U") or the R_i (which = "R")."""
    L = c + N - 2
    worst = 0.0
    for trial in range(trials):
        idx = trial % N
        E = rng.standard_normal((c, c) if which == "U" else (L + 1, c))
        E /= np.linalg.norm(E)

        def perturb(U_, R_, t, idx=idx, E=E):
            if which == "U":
                return [u + (t * E if k == idx else 0) for k, u in enumerate(U_)], R_
            return U_, [r + (t * E if k == idx else 0) for k, r in enumerate(R_)]
        slope, rise, _ = _phi_slope_and_rise(U, R, perturb)
        assert rise > 0
        worst = max(worst, abs(slope))
    return worst


def test_als_loop_holds_the_pairs_it_reports_and_takes_its_steps_in_order():
    """The iteration of Sec. II-D as a whole (the single steps are pinned above): every entry of the
    reported history is Phi of the pair held at that point, evaluated here from the M_i matrices; in
    every iteration the unprojected U minimises Phi for the R of the iteration BEFORE (zero slope in U
    there, and a clearly non-zero one for the new R, which rules out a swapped order), the new U is its
    nearest point with singular values in [a0, b0] (Mirsky's bound attained), and the new R minimises
    Phi for the projected U (zero slope in R; in particular the last R was refitted after the last
    projection)."""
    N, c, C = 3, 5, 1e2
    des = Dz.kappa_constrained(N, c, C, _rng_B(N, c, 3), iters=6, tol=0.0, keep_pairs=True)
    info = des.info
    pairs, U_ls, hist = info["pairs"], info["U_ls"], info["phi_history"]
    a0, b0 = info["a0"], info["b0"]
    assert len(pairs) == len(hist) == info["iters_done"] + 1 == 7 and len(U_ls) == 6
    for (U, R), ph in zip(pairs, hist):
        assert P.phi(U, R) == pytest.approx(ph, rel=1e-12)
    assert P.phi(des.U, des.R) == pytest.approx(hist[-1], rel=1e-12)
    for a, b in zip(pairs[-1][0], des.U):
        assert np.array_equal(a, b)
    for a, b in zip(pairs[-1][1], des.R):
        assert np.array_equal(a, b)
    rng = np.random.default_rng(8)
    for t in range(1, len(pairs)):
        (U_prev, R_prev), (U_new, R_new), V = pairs[t - 1], pairs[t], U_ls[t - 1]
        scale = max(1.0, hist[t - 1])
        assert _max_slope(V, R_prev, "U", rng, N, c) < 1e-6 * scale          # U-step used the previous R
        assert _max_slope(V, R_new, "U", rng, N, c) > 1e-4 * scale            # ... and not the new one
        for k in range(N):                                                    # projection of exactly that V
            sV = np.linalg.svd(V[k], compute_uv=False)
            sU = np.linalg.svd(U_new[k], compute_uv=False)
            assert sU[-1] >= a0 * (1 - 1e-10) and sU[0] <= b0 * (1 + 1e-10)
            assert np.linalg.norm(V[k] - U_new[k]) == pytest.approx(np.linalg.norm(sV - np.clip(sV, a0, b0)),
                                                                     rel=1e-8, abs=1e-12)
        assert _max_slope(U_new, R_new, "R", rng, N, c) < 1e-6 * scale        # R-step after the projection
        assert P.phi(V, R_prev) == pytest.approx(info["steps"][t - 1][1], rel=1e-12)
    # the start: the projected epsilon-construction with its least-squares decoder
    U0, R0 = pairs[0]
    init = Dz.epsilon(N, c, info["eps_init"], _rng_B(N, c, 3))
    assert a0 == pytest.approx(min(np.linalg.svd(u, compute_uv=False)[-1] for u in init.U), rel=1e-12)
    for k in range(N):
        sI = np.linalg.svd(init.U[k], compute_uv=False)
        assert np.linalg.norm(init.U[k] - U0[k]) == pytest.approx(np.linalg.norm(sI - np.clip(sI, a0, b0)), rel=1e-8)
    assert _max_slope(U0, R0, "R", rng, N, c) < 1e-6 * max(1.0, hist[0])


def test_als_end_point_is_a_fixed_point_up_to_its_stopping_rule():
    """When the run stops on its tolerance, one more iteration from the returned pair changes Phi by
    about the tolerance and moves U and R by a step of the same small order (the heuristic converges
    sublinearly: measured 3e-5 relative here), so what is returned is the loop's own fixed point and
    not a pair from somewhere inside an iteration.  A run cut off by the iteration cap says so."""
    N, c, C, tol = 3, 7, 1e2, 1e-6
    B = _rng_B(N, c, 5)
    des = Dz.kappa_constrained(N, c, C, B, iters=4000, tol=tol)
    assert des.info["stopped_on_tol"] and des.info["iters_done"] < 4000
    hist = des.info["phi_history"]
    assert abs(hist[-2] - hist[-1]) <= tol * hist[-1]
    assert all(abs(a - b) > tol * b for a, b in zip(hist[:-2], hist[1:-1]))       # it did not stop earlier
    _, U2, R2 = Dz.als_iteration(des.U, des.R, des.info["a0"], des.info["b0"], N, c)
    ph2 = P.phi(U2, R2)
    assert abs(ph2 - hist[-1]) <= 2 * tol * hist[-1]
    for k in range(N):
        assert np.linalg.norm(U2[k] - des.U[k]) <= 2e-4 * np.linalg.norm(des.U[k])
        assert np.linalg.norm(R2[k] - des.R[k]) <= 2e-4 * np.linalg.norm(des.R[k])
    short = Dz.kappa_constrained(N, c, C, B, iters=5, tol=tol)
    assert not short.info["stopped_on_tol"] and short.info["iters_done"] == 5


def test_kappa_constrained_interval_comes_from_the_initial_design():
    """[a0, b0] of Sec. II-D: a0 = the smallest singular value over the encoders of the initial
    epsilon-construction, b0 = a0 C / sqrt(N).  Pinned to a 120-digit SVD of those encoders, which at
    N = 4, c = 24 have condition numbers beyond 1e10, where an fp64 SVD of U_k would already lose digits."""
    import mpmath as mp
    N, c, C = 4, 24, 1e4
    B = _rng_B(N, c, 2)
    des = Dz.kappa_constrained(N, c, C, B, iters=1)
    init = Dz.epsilon(N, c, des.info["eps_init"], B)
    with mp.workdps(120):
        smallest = min(min(mp.svd_r(Um, compute_uv=False)) for Um in init.U_mp)
    assert des.info["a0"] == pytest.approx(float(smallest), rel=1e-12)
    assert des.info["b0"] == pytest.approx(float(smallest) * C / np.sqrt(N), rel=1e-12)
    assert max(P.kappa2(u) for u in init.U) > 1e10


def test_surrogate_is_well_conditioned():
    des = Dz.custom_orthogonal(4, 8, np.random.default_rng(0))
    for u in des.U:
        assert P.kappa2(u) == pytest.approx(1.0, abs=1e-9)


@pytest.mark.parametrize("N,C", [(3, 1e6), (4, 1e4)])
def test_kappa_constrained_reaches_the_known_optimum_when_c_equals_N(N, C):
    """c = N is the exactly solvable case (Lemma 1 only forbids Phi = 0 for c > N; the classic
    ring all-reduce is an exact solution): with a loose bound the constrained problem has
    optimum Phi = 0 wherever the projection interval [a0, b0] does not bind (true for this B),
    and the heuristic must get there from its O(eps^2) start, with the decoded sum exact."""
    c = N
    B = _rng_B(N, c, 12)
    des = Dz.kappa_constrained(N, c, C, B, iters=1000, tol=1e-30)
    hist = des.info["phi_history"]
    assert hist[0] > 1e-4 and hist[-1] < 1e-18
    assert max(P.kappa2(P.m_matrix(des.U, i)) for i in range(N)) <= C
    rng = np.random.default_rng(0)
    g = [rng.standard_normal(c * 5) for _ in range(N)]
    res = P.allreduce(g, des.U, des.R, 1.0)
    for i in range(N):
        assert P.rel_l2(res["out"][i], P.exact_sum(g)) < 1e-9
