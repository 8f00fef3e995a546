"""Pins for oracle.protocol: what the paper and plain linear algebra fix."""
import itertools
import os

import numpy as np
import pytest

from oracle import designs as Dz
from oracle import protocol as P


def _onehot_deltas(N, c):
    """delta_{i,j} = unit vector e_{i*c + (j-1)} in R^{N c}: every message is
    then a 0/1 (or signed) indicator of which deltas it contains."""
    p = N * c
    Delta = []
    for i in range(N):
        M = np.zeros((p, c))
        for j in range(c):
            M[i * c + j, j] = 1.0
        Delta.append(M)
    return Delta


def _vec(terms, N, c):
    v = np.zeros(N * c)
    for w, j in terms:
        v[w * c + (j - 1)] += 1.0
    return v


def _parse_terms(s):
    return [tuple(int(t) for t in tok.split(",")) for tok in s.split()]


def test_fig1_messages_and_states(golden_dir):
    N, c = 4, 5
    _, _, tr = P.run_rounds(_onehot_deltas(N, c), trace=True)
    checked = 0
    for line in open(os.path.join(golden_dir, "fig1_n4_c5.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = [s.strip() for s in line.split("=")]
        kind, i, k = lhs.split()
        i, k = int(i), int(k)
        if kind == "x":
            np.testing.assert_array_equal(tr["x"][k][i], _vec(_parse_terms(rhs), N, c))
        elif kind == "sigma_terms":
            np.testing.assert_array_equal(tr["sigma"][k][i], _vec(_parse_terms(rhs), N, c))
        elif kind == "sigma":
            t = rhs.split()
            assert t[0] == "x" and t[3] == "-"
            w, kk = int(t[1]), int(t[2])
            expect = tr["x"][kk][w] - _vec(_parse_terms(t[4]), N, c)
            np.testing.assert_array_equal(tr["sigma"][k][i], expect)
        else:
            raise AssertionError(kind)
        checked += 1
    assert checked == 23


def test_m_matrix_printed_pattern(golden_dir):
    N, c = 4, 5
    # U_w[:, j-1] tagged with the number 10*w + j everywhere in the column
    U = [np.tile(10 * w + np.arange(1, c + 1, dtype=float), (c, 1)) for w in range(N)]
    Y, _, _ = P.run_rounds(_onehot_deltas(N, c))
    for line in open(os.path.join(golden_dir, "m_pattern_n4_c5.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = [s.strip() for s in line.replace(" : ", " = ").split("=")]
        t = lhs.split()
        if t[0] == "M":
            i, r = int(t[1]), int(t[2])
            blk = P.m_matrix(U, i)[r * c:(r + 1) * c, :]
            toks = rhs.split()
            assert len(toks) == N + c - 1
            for col, tok in enumerate(toks):
                if tok == ".":
                    assert np.all(blk[:, col] == 0)
                else:
                    w, j = (int(v) for v in tok.split(","))
                    assert np.all(blk[:, col] == 10 * w + j)
        else:   # "y i m = terms": column m of Y_i from the protocol itself
            i, m = int(t[1]), int(t[2])
            np.testing.assert_array_equal(Y[i][:, m - 1], _vec(_parse_terms(rhs), N, c))


@pytest.mark.parametrize("N,c", [(2, 2), (2, 5), (3, 3), (3, 7), (4, 5), (4, 9), (5, 5), (5, 8)])
def test_rounds_equal_composed_map_for_arbitrary_U(N, c):
    """Y_i = G^(i) M_i(U) for any encoders (not only MPC designs)."""
    rng = np.random.default_rng(100 * N + c)
    p = 3
    U = [rng.standard_normal((c, c)) for _ in range(N)]
    g = [rng.standard_normal(c * p) for _ in range(N)]
    G = [P.chunk_matrix(x, c) for x in g]
    Delta = [P.encode(G[i], U[i]) for i in range(N)]
    for literal in (False, True):
        Y, sent, _ = P.run_rounds(Delta, literal_store=literal)
        for i in range(N):
            # brute force, entry by entry, straight from the block structure of M_i
            L = c + N - 2
            for q in range(p):
                for m in range(L + 1):
                    acc = 0.0
                    for r in range(N):
                        col = m - (N - 1 - r)
                        if 0 <= col < c:
                            w = (i + r) % N
                            acc += sum(G[w][q, l] * U[w][l, col] for l in range(c))
                    assert abs(Y[i][q, m] - acc) < 1e-10
            np.testing.assert_allclose(Y[i], P.stacked_gradients(G, i) @ P.m_matrix(U, i), atol=1e-10)
        assert sent == [(c + N - 2) * p] * N


def test_whole_pipeline_is_one_linear_map():
    rng = np.random.default_rng(7)
    N, c, p = 4, 6, 4
    L = c + N - 2
    U = [rng.standard_normal((c, c)) for _ in range(N)]
    R = [rng.standard_normal((L + 1, c)) for _ in range(N)]
    g = [rng.standard_normal(c * p) for _ in range(N)]
    G = [P.chunk_matrix(x, c) for x in g]
    res = P.allreduce(g, U, R, scale=0.25)
    for i in range(N):
        Ghat = 0.25 * P.stacked_gradients(G, i) @ (P.m_matrix(U, i) @ R[i])
        np.testing.assert_allclose(res["out"][i], P.unchunk(Ghat), atol=1e-10)


@pytest.mark.parametrize("N,c", [(3, 4), (4, 5), (4, 12), (6, 7)])
def test_message_closed_form(N, c):
    """x_{i,k} = sum_{t=0}^{N-1} delta_{i-t, k-t}, delta_{.,j} = 0 outside 1..c
    (unrolling Eq. update_eqns)."""
    _, _, tr = P.run_rounds(_onehot_deltas(N, c), trace=True)
    L = c + N - 2
    for k in range(1, L + 1):
        for i in range(N):
            terms = [((i - t) % N, k - t) for t in range(N) if 1 <= k - t <= c]
            np.testing.assert_array_equal(tr["x"][k][i], _vec(terms, N, c))


def test_literal_and_direct_store_agree():
    rng = np.random.default_rng(3)
    N, c, p = 5, 9, 8
    Delta = [rng.standard_normal((p, c)) for _ in range(N)]
    Ya, _, _ = P.run_rounds(Delta, literal_store=True)
    Yb, _, _ = P.run_rounds(Delta, literal_store=False)
    for a, b in zip(Ya, Yb):
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


@pytest.mark.parametrize("N,c,p", [(4, 8, 8192), (4, 16, 1048576), (8, 32, 44207744), (8, 64, 4194304), (16, 128, 1 << 23)])
def test_rates_are_exact(N, c, p):
    """Communication rate 1+(N-2)/c and storage rate 1+N/c as exact integer
    identities (Sec. II-B)."""
    d = c * p
    L = P.num_rounds(N, c)
    sent = L * p
    stored = (c + N) * p
    assert sent * c == d * (c + N - 2)
    assert stored * c == d * (c + N)
    comm, stor = P.rates(N, c)
    assert comm == pytest.approx(1 + (N - 2) / c) and stor == pytest.approx(1 + N / c)


def test_counters_from_the_run():
    rng = np.random.default_rng(0)
    N, c, p = 4, 8, 5
    U = [rng.standard_normal((c, c)) for _ in range(N)]
    R = [rng.standard_normal((c + N - 1, c)) for _ in range(N)]
    res = P.allreduce([rng.standard_normal(c * p) for _ in range(N)], U, R)
    d = c * p
    assert all(s * c == d * (c + N - 2) for s in res["values_sent_per_worker"])
    assert res["values_stored_per_worker"] * c == d * (c + N)
    assert res["rounds"] == c + N - 2


def test_chunking_layout():
    c, p = 3, 4
    g = np.arange(c * p, dtype=float)
    G = P.chunk_matrix(g, c)
    assert G.shape == (p, c)
    for l in range(c):
        np.testing.assert_array_equal(G[:, l], g[l * p:(l + 1) * p])
    np.testing.assert_array_equal(P.unchunk(G), g)
    with pytest.raises(ValueError):
        P.chunk_matrix(np.zeros(10), 3)


def test_classic_ring_case_is_exact():
    """c = N with D = I: Phi = 0, the output is the exact sum and the round
    count is the basic ring all-reduce's 2(N-1)."""
    rng = np.random.default_rng(11)
    for N in (2, 3, 4, 6):
        c = N
        B = rng.standard_normal((N, c))
        des = Dz.epsilon(N, c, 0.0, B)
        assert des.L == 2 * (N - 1)
        g = [rng.standard_normal(c * 6) for _ in range(N)]
        res = P.allreduce(g, des.U, des.R)
        for i in range(N):
            assert P.rel_l2(res["out"][i], P.exact_sum(g)) < 1e-12
        assert P.phi(des.U, des.R) < 1e-20


def test_per_worker_closed_form():
    """From Prop. 1: G_hat_i = sum_{j>=i} G_j + (sum_{j<i} G_j) D^{-1}; worker 0
    is exact, worker i carries i perturbed terms."""
    rng = np.random.default_rng(5)
    N, c, p, eps = 4, 7, 5, 1e-2
    B = rng.standard_normal((N, c))
    des = Dz.epsilon(N, c, eps, B)
    Dinv = np.diag([1.0 / (1.0 + eps * h) for h in Dz.default_h(c)])
    g = [rng.standard_normal(c * p) for _ in range(N)]
    G = [P.chunk_matrix(x, c) for x in g]
    res = P.allreduce(g, des.U, des.R)
    for i in range(N):
        expect = sum(G[j] for j in range(i, N))
        if i > 0:
            expect = expect + sum(G[j] for j in range(i)) @ Dinv
        np.testing.assert_allclose(res["out"][i], P.unchunk(expect), atol=1e-8)
    assert P.rel_l2(res["out"][0], P.exact_sum(g)) < 1e-9


def test_error_identity_and_bound():
    """|| g_hat_i - sum || = || G^(i) (M_i R_i - T) ||_F <= ||G^(i)||_2 delta_dec
    (Eq. bounded_spectral_assumption)."""
    rng = np.random.default_rng(9)
    N, c, p = 4, 6, 10
    des = Dz.epsilon(N, c, 5e-2, rng.standard_normal((N, c)))
    g = [rng.standard_normal(c * p) for _ in range(N)]
    G = [P.chunk_matrix(x, c) for x in g]
    res = P.allreduce(g, des.U, des.R)
    T = P.target(N, c)
    for i in range(N):
        E = P.m_matrix(des.U, i) @ des.R[i] - T
        Gi = P.stacked_gradients(G, i)
        lhs = np.linalg.norm(res["out"][i] - P.exact_sum(g))
        assert lhs == pytest.approx(np.linalg.norm(Gi @ E, "fro"), rel=1e-6, abs=1e-9)
        assert lhs <= np.linalg.norm(Gi, 2) * np.linalg.norm(E, "fro") * (1 + 1e-9) + 1e-9


def test_randomised_shapes_composed_map_and_prop1():
    """Seeded random (N, c, p): rounds == G^(i) M_i(U) for random encoders, the decoded
    output is the one linear map G^(i) (M_i R_i), and for an epsilon design worker 0
    recovers the exact sum (Prop. 1 with i = 0)."""
    rng = np.random.default_rng(2024)
    for _ in range(25):
        N = int(rng.integers(2, 7))
        c = int(rng.integers(N, N + 9))
        p = int(rng.integers(1, 6))
        L = c + N - 2
        U = [rng.standard_normal((c, c)) for _ in range(N)]
        R = [rng.standard_normal((L + 1, c)) for _ in range(N)]
        g = [rng.standard_normal(c * p) for _ in range(N)]
        G = [P.chunk_matrix(x, c) for x in g]
        res = P.allreduce(g, U, R, 0.5)
        for i in range(N):
            Gi = P.stacked_gradients(G, i)
            np.testing.assert_allclose(res["Y"][i], Gi @ P.m_matrix(U, i), atol=1e-9)
            np.testing.assert_allclose(res["out"][i], P.unchunk(0.5 * Gi @ (P.m_matrix(U, i) @ R[i])), atol=1e-9)
        assert res["values_sent_per_worker"] == [L * p] * N
        des = Dz.epsilon(N, c, 0.03, rng.standard_normal((N, c)))
        out = P.allreduce(g, des.U, des.R)["out"]
        assert P.rel_l2(out[0], P.exact_sum(g)) < 1e-7
