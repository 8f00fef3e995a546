"""Coefficient constructions for CERAR, written from the paper's definitions.

Test infrastructure only (see the package docstring).  The multiplicative
perturbation construction (MPC) and its two instances are evaluated with
mpmath at high working precision and then rounded to fp64: the windows
A_l are extremely ill-conditioned by design (Remark after Theorem 1,
Corollary 1), so a plain fp64 inverse would not be a trustworthy reference.
The condition-number-constrained design is an fp64 iteration (numpy).

kappa_constrained: every step of an iteration is pinned to the property that defines
it (the U-step and the R-step are stationary minimisers of the brute-force Phi, the
projection is the Frobenius-nearest matrix with singular values in the interval), the
loop is pinned to the order of its steps and to the pairs it reports (every history entry
is Phi of the pair held then; the returned pair is a fixed point up to the stopping rule),
and for c = N, where the optimum Phi = 0 is known, it is checked to reach it.  PARITY
UNPINNED for the end point at c > N only: which local solution the heuristic reaches has no
published counterpart (the paper prints no U, R or Phi for it).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import mpmath as mp
import numpy as np

from . import protocol

DEFAULT_DPS = 120


@dataclass
class Design:
    N: int
    c: int
    U: list                 # N arrays c x c, fp64
    R: list                 # N arrays (L+1) x c, fp64
    kind: str = "custom"
    U_mp: list | None = None    # high-precision copies (MPC designs only)
    R_mp: list | None = None
    Dmat_mp: object | None = None
    info: dict = field(default_factory=dict)

    @property
    def L(self):
        return protocol.num_rounds(self.N, self.c)


def _to_np(M) -> np.ndarray:
    return np.array([[float(M[i, j]) for j in range(M.cols)] for i in range(M.rows)], dtype=np.float64)


def _is_vector(D) -> bool:
    return isinstance(D, (list, tuple)) or (isinstance(D, np.ndarray) and D.ndim == 1)


def mpc_sequence(B, D, N: int, c: int, lo: int, hi: int, dps: int = DEFAULT_DPS):
    """Rows a_l for l in [lo, hi]: a_{r+mN} = b_r D^m for every integer m,
    negative m included (Eq. a_seq).  B is N x c; D is either the diagonal of a
    diagonal matrix (length-c vector) or a full c x c matrix.  Returns a dict
    l -> 1 x c mp.matrix."""
    with mp.workdps(dps):
        Bm = mp.matrix(B) if not isinstance(B, mp.matrix) else B
        rows = {}
        if _is_vector(D):
            dv = [mp.mpf(x) for x in D]
            for l in range(lo, hi + 1):
                m, r = divmod(l, N)            # floor division: r in [0, N)
                rows[l] = mp.matrix([[Bm[r, j] * dv[j] ** m for j in range(c)]])
        else:
            Dm = mp.matrix(D) if not isinstance(D, mp.matrix) else D
            Dinv = mp.inverse(Dm)
            m_lo, m_hi = lo // N, hi // N
            powers = {0: mp.eye(c)}
            for m in range(1, m_hi + 1):
                powers[m] = powers[m - 1] * Dm
            for m in range(-1, m_lo - 1, -1):
                powers[m] = powers[m + 1] * Dinv
            for l in range(lo, hi + 1):
                m, r = divmod(l, N)
                rows[l] = Bm[r, :] * powers[m]
        return rows


def _stack(rows, l0: int, n: int, c: int):
    A = mp.matrix(n, c)
    for t in range(n):
        for j in range(c):
            A[t, j] = rows[l0 + t][0, j]
    return A


def mpc(B, D, N: int, c: int, dps: int = DEFAULT_DPS, kind: str = "mpc") -> Design:
    """Multiplicative perturbation construction (Sec. II-B.1):
    A_l = [a_l; ...; a_{l+c-1}] (Eq. A-ell), V_{N-1-k} = A_k, U_k = V_k^{-1}
    (Eq. encoders), R_i[l, :] = a_{l-i}, l = 0..L (Eq. decoderconstruction)."""
    L = protocol.num_rounds(N, c)
    with mp.workdps(dps):
        rows = mpc_sequence(B, D, N, c, -(N - 1), L + c, dps)
        U_mp = [None] * N
        for k in range(N):
            A_k = _stack(rows, k, c, c)
            U_mp[N - 1 - k] = mp.inverse(A_k)      # U_{N-1-k} = V_{N-1-k}^{-1} = A_k^{-1}
        R_mp = [_stack(rows, -i, L + 1, c) for i in range(N)]
        if _is_vector(D):
            Dm = mp.diag([mp.mpf(x) for x in D])
        else:
            Dm = mp.matrix(D)
        U = [_to_np(M) for M in U_mp]
        R = [_to_np(M) for M in R_mp]
    return Design(N, c, U, R, kind, U_mp, R_mp, Dm)


def default_xi(c: int):
    """Equally spaced distinct reals in [-1, 1] (the paper leaves xi_j free)."""
    if c == 1:
        return [0.0]
    return [-1.0 + 2.0 * j / (c - 1) for j in range(c)]


def vandermonde(N: int, c: int, tau: float, xi=None, dps: int = DEFAULT_DPS) -> Design:
    """Vandermonde construction (Sec. II-B.2): z_j = exp(tau xi_j),
    b_l = [z_1^l .. z_c^l], D_tau = diag(z_j^N)."""
    xi = default_xi(c) if xi is None else list(xi)
    with mp.workdps(dps):
        z = [mp.exp(mp.mpf(tau) * mp.mpf(x)) for x in xi]
        B = mp.matrix(N, c)
        for l in range(N):
            for j in range(c):
                B[l, j] = z[j] ** l
        Dv = [zj ** N for zj in z]
        des = mpc(B, Dv, N, c, dps, "vandermonde")
    des.info.update(tau=tau, xi=xi)
    return des


def default_h(c: int):
    """Diagonal of H: equally spaced in [-1, 1], so ||H||_2 = 1 and the
    entries are distinct (the paper asks for a diagonal H with small entries
    after scaling by epsilon)."""
    return default_xi(c)


def epsilon(N: int, c: int, eps: float, B, h=None, dps: int = DEFAULT_DPS) -> Design:
    """epsilon-construction (Sec. II-C): D_eps = I + eps H, here with diagonal
    H = diag(h), and a given N x c base matrix B (i.i.d. N(0,1) in the paper's
    experiments; it is an input here)."""
    h = default_h(c) if h is None else list(h)
    with mp.workdps(dps):
        Bm = mp.matrix(np.asarray(B, dtype=np.float64).tolist())
        Dv = [1 + mp.mpf(eps) * mp.mpf(x) for x in h]
        des = mpc(Bm, Dv, N, c, dps, "epsilon")
    des.info.update(eps=eps, h=h)
    return des


# ---------------------------------------------------------- high-precision diagnostics

def phi_mp(des: Design, dps: int = DEFAULT_DPS):
    """Phi(U, R) evaluated in high precision (the fp64 product M_i R_i loses
    everything to cancellation for ill-conditioned designs)."""
    N, c, L = des.N, des.c, des.L
    with mp.workdps(dps):
        tot = mp.mpf(0)
        for i in range(N):
            for r in range(N):
                Uk = des.U_mp[(i + r) % N]
                s = N - 1 - r
                W = des.R_mp[i][s:s + c, :]
                E = Uk * W - mp.eye(c)
                tot += sum(E[a, b] ** 2 for a in range(c) for b in range(c))
        return tot


def block_products_mp(des: Design, dps: int = DEFAULT_DPS):
    """All blocks U_{i-1-s} W_s(R_i), as a dict (i, s) -> mp.matrix."""
    N, c = des.N, des.c
    out = {}
    with mp.workdps(dps):
        for i in range(N):
            for s in range(N):
                out[(i, s)] = des.U_mp[(i - 1 - s) % N] * des.R_mp[i][s:s + c, :]
    return out


def finite_difference_matrix(n: int) -> np.ndarray:
    """F_n: lower triangular, entry (j, k) = (-1)^(j-k) binom(j, k), 0-based
    (Appendix, finite-difference factorisation)."""
    from math import comb
    F = np.zeros((n, n), dtype=np.int64)
    for j in range(n):
        for k in range(j + 1):
            F[j, k] = (-1) ** (j - k) * comb(j, k)
    return F


def window_mp(B, Dv, N: int, c: int, l: int, dps: int = DEFAULT_DPS):
    """A_l for a diagonal D given by its diagonal Dv."""
    with mp.workdps(dps):
        rows = mpc_sequence(B, Dv, N, c, l, l + c - 1, dps)
        return _stack(rows, l, c, c)


def singular_values_mp(A, dps: int = DEFAULT_DPS):
    with mp.workdps(dps):
        S = mp.svd_r(A, compute_uv=False)
        return sorted([S[i] for i in range(len(S))], reverse=True)


def k_limit(B, h, N: int, c: int, l: int) -> np.ndarray:
    """K^(l)(B, H), H = diag(h): the eps -> 0 limit of K_l(eps) in the factorisation
    F~_l Pi_l A_l(eps) = Lambda_l(eps) K_l(eps) (Sec. II-C).  With c = beta N + s it
    stacks B, BH, .., BH^(beta-1) and, if s > 0, the rows E_l = {l, .., l+s-1} mod N of
    BH^beta."""
    B = np.asarray(B, dtype=np.float64)
    h = np.asarray(h, dtype=np.float64)
    beta, s = divmod(c, N)
    blocks = [B * h ** j for j in range(beta)]
    if s > 0:
        E = [(l + t) % N for t in range(s)]
        blocks.append((B * h ** beta)[E, :])
    return np.concatenate(blocks, axis=0)


def gamma(B, h, N: int, c: int) -> float:
    """min over l = 0..N-1 of sigma_min(K^(l)(B, H)): the constant the analysis of the
    epsilon-construction assumes positive (the Assumption of Sec. II-C)."""
    return min(float(np.linalg.svd(k_limit(B, h, N, c, l), compute_uv=False)[-1]) for l in range(N))


def optimize_h(B, N: int, c: int, h0=None, sweeps: int = 2, grid: int = 17):
    """A deterministic choice of the diagonal H from B.  The paper only mentions that H can be derived
    deterministically from B, without a rule (appendix on the numerical experiments), and that the
    analysis needs gamma(B, H) > 0 (Sec. II-C); the reading taken here is coordinate ascent on gamma:
    start from h0 (default: equally spaced in [-1, 1]); visit the coordinates j = 0..c-1 in order; for
    each, try the `grid` equally spaced values of [-1, 1] in increasing order and move h_j to the first
    value that gives the largest gamma, if that is larger than the current one (by more than 1e-12
    relative) and leaves max|h| = 1 (so that ||H||_2 = 1 stays comparable between choices); stop after
    `sweeps` passes or a pass without a move.  Returns (h, gamma(B, h), moves)."""
    B = np.asarray(B, dtype=np.float64)
    h = np.array(default_h(c) if h0 is None else h0, dtype=np.float64)
    h = h / np.abs(h).max()
    cand = [-1.0 + 2.0 * t / (grid - 1) for t in range(grid)]
    best = gamma(B, h, N, c)
    moves = 0
    for _ in range(sweeps):
        moved = False
        for j in range(c):
            keep, best_j, val_j = h[j], None, best
            for g in cand:
                if g == keep:
                    continue
                h[j] = g
                if np.abs(h).max() < 1.0:
                    continue
                v = gamma(B, h, N, c)
                if v > val_j * (1 + 1e-12):
                    val_j, best_j = v, g
            h[j] = keep if best_j is None else best_j
            if best_j is not None:
                best, moved, moves = val_j, True, moves + 1
        if not moved:
            break
    return h, best, moves


# ---------------------------------------------------------- kappa-constrained design

def _ls_R(U, N, c):
    T = protocol.target(N, c)
    return [np.linalg.lstsq(protocol.m_matrix(U, i), T, rcond=None)[0] for i in range(N)]


def _ls_U(R, N, c):
    # Phi = sum_i sum_s || U_{i-1-s} W_s(R_i) - I ||_F^2 (block form used in the
    # proof of Lemma 1).  For fixed k the blocks with i-1-s = k (mod N) give
    # U_k [W_{s_0}(R_0) .. W_{s_{N-1}}(R_{N-1})] ~ [I .. I], s_i = (i-1-k) mod N.
    U = []
    for k in range(N):
        P = np.concatenate([protocol.window(R[i], (i - 1 - k) % N, c) for i in range(N)], axis=1)
        Tk = np.concatenate([np.eye(c)] * N, axis=1)
        Uk_T = np.linalg.lstsq(P.T, Tk.T, rcond=None)[0]
        U.append(Uk_T.T)
    return U


def _project(U, a0, b0):
    out = []
    for Uk in U:
        X, s, Zt = np.linalg.svd(Uk)
        out.append((X * np.clip(s, a0, b0)) @ Zt)
    return out


def als_iteration(U, R, a0: float, b0: float, N: int, c: int):
    """One iteration of the heuristic of Sec. II-D from the pair (U, R): minimise Phi over U with R
    fixed, project the singular values of every U_k into [a0, b0], minimise Phi over R with the
    projected U fixed.  Returns (U_ls, U_new, R_new): the unprojected minimiser, and the new pair."""
    U_ls = _ls_U(R, N, c)
    U_new = _project(U_ls, a0, b0)
    R_new = _ls_R(U_new, N, c)
    return U_ls, U_new, R_new


def kappa_constrained(N: int, c: int, kappa_max: float, B, h=None, eps_init: float = 0.1,
                      iters: int = 200, tol: float = 1e-6, dps: int = DEFAULT_DPS,
                      keep_pairs: bool = False) -> Design:
    """Alternating least-squares heuristic for
        minimise Phi(U, R)  s.t.  kappa_2(M_i(U)) <= C        (Eq. F)
    as Sec. II-D describes it: start from the epsilon-construction; in one
    iteration minimise over R with U fixed, then over U with R fixed, then
    project the singular values of every U_k into a common interval [a0, b0]
    with sqrt(N) b0 / a0 <= C.  Choices the paper leaves open (documented as
    readings): eps_init = 0.1, a0 = min_k sigma_min(U_k of the initial design),
    b0 = a0 C / sqrt(N), stop after `iters` iterations or when Phi changes by
    less than tol (relative), and a last R-step after the last projection
    (so the pair returned is always (projected U, its least-squares R)).
    keep_pairs: also keep, in info["pairs"], every pair (U, R) the iteration held
    and, in info["U_ls"], the unprojected U of every iteration (for the tests)."""
    init = epsilon(N, c, eps_init, B, h, dps)
    U = [u.copy() for u in init.U]
    # sigma_min(U_k) = 1 / sigma_max(U_k^{-1}): the initial encoders have condition numbers up to
    # 1e15 (Corollary 1), where an fp64 SVD of U_k itself gets its smallest singular value wrong in
    # the fourth digit; the inverse (a window A_l, exact in the high-precision design) has it as its
    # LARGEST singular value, which fp64 delivers to full accuracy
    with mp.workdps(dps):
        inv_norms = [np.linalg.svd(_to_np(mp.inverse(Um)), compute_uv=False)[0] for Um in init.U_mp]
    a0 = float(min(1.0 / s for s in inv_norms))
    b0 = a0 * kappa_max / np.sqrt(N)
    U = _project(U, a0, b0)
    R = _ls_R(U, N, c)
    hist = [protocol.phi(U, R)]
    steps = []
    pairs, unprojected = [(U, R)], []
    done = 0
    stopped_on_tol = False
    for it in range(iters):
        U_ls, U, R_next = als_iteration(U, R, a0, b0, N, c)
        phi_after_U = protocol.phi(U_ls, R)
        R = R_next
        cur = protocol.phi(U, R)
        steps.append((hist[-1], phi_after_U, cur))
        hist.append(cur)
        if keep_pairs:
            pairs.append((U, R))
            unprojected.append(U_ls)
        done = it + 1
        if abs(hist[-2] - cur) <= tol * max(cur, 1e-300):
            stopped_on_tol = True
            break
    des = Design(N, c, U, R, "kappa")
    des.info.update(kappa_max=kappa_max, a0=a0, b0=b0, phi_history=hist, steps=steps,
                    iters_done=done, eps_init=eps_init, stopped_on_tol=stopped_on_tol)
    if keep_pairs:
        des.info.update(pairs=pairs, U_ls=unprojected)
    return des


def custom_orthogonal(N: int, c: int, rng: np.random.Generator) -> Design:
    """Well-conditioned surrogate coefficients (random orthogonal U_i, Gaussian
    R_i with variance 1/(L+1)).  Not a CERAR design: the kernels do not care
    what the numbers mean, and with kappa ~ 1 a data-path bug cannot hide
    under rounding noise."""
    L = protocol.num_rounds(N, c)
    U = [np.linalg.qr(rng.standard_normal((c, c)))[0] for _ in range(N)]
    R = [rng.standard_normal((L + 1, c)) / np.sqrt(L + 1) for _ in range(N)]
    return Design(N, c, U, R, "surrogate")
