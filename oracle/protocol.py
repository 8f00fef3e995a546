"""CERAR data path in plain numpy fp64, step by step as the paper states it.

Test infrastructure only (see the package docstring).  Notation follows the
paper: N workers W_0..W_{N-1} on a clockwise ring, c chunks per gradient,
p = d / c, L = c + N - 2 rounds, encoders U_i (c x c), decoders R_i
((L+1) x c), encoded vectors delta_{i,j}, messages x_{i,k}, rolling state
sigma_{i,k}, buffers D_{i,j}, B_{i,j}, C_i, observations Y_i.
"""
from __future__ import annotations

import numpy as np


def num_rounds(N: int, c: int) -> int:
    """L = c + N - 2 (Sec. II, first paragraph)."""
    return c + N - 2


def chunk_matrix(g: np.ndarray, c: int) -> np.ndarray:
    """G_i in R^{p x c}: column l is chunk g_i[l] = g[l*p:(l+1)*p] (Sec. II,
    definition of G_i).  The paper assumes c | d (zero-padding otherwise)."""
    g = np.asarray(g, dtype=np.float64)
    d = g.shape[0]
    if d % c != 0:
        raise ValueError("c must divide d (the caller zero-pads)")
    p = d // c
    return g.reshape(c, p).T.copy()


def unchunk(G: np.ndarray) -> np.ndarray:
    """Inverse of chunk_matrix: stack the columns of a p x c matrix."""
    return np.asarray(G, dtype=np.float64).T.reshape(-1).copy()


def encode(G: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Delta_i = G_i U_i (Sec. II, 'Initialization')."""
    return np.asarray(G, np.float64) @ np.asarray(U, np.float64)


def run_rounds(Delta, *, literal_store: bool = False, trace: bool = False):
    """Algorithm 1, for all N workers concurrently.

    Delta : list of N arrays (p x c); column j-1 is delta_{i,j}.
    literal_store : if True the received vector is stored exactly as the
        algorithm prints it (C <- C - D_j ; D_j <- D_j + C); otherwise the
        received vector is written to D_j directly.  The two agree up to
        rounding.
    trace : also return the messages x[k][i] and the states sigma[k][i].

    Returns (Y, sent, extra): Y[i] is the p x (L+1) observation matrix
    [B_{i,1} .. B_{i,N-1} | D_{i,1} .. D_{i,c}], sent[i] the number of real
    values worker i transmitted, extra a dict with the trace (or empty).
    """
    N = len(Delta)
    p, c = Delta[0].shape
    L = num_rounds(N, c)
    # buffers of worker i: D[i][j-1], B[i][k-1], C[i]
    D = [[np.array(Delta[i][:, j], dtype=np.float64) for j in range(c)] for i in range(N)]
    B = [[None] * (N - 1) for _ in range(N)]
    C = [np.zeros(p, dtype=np.float64) for _ in range(N)]   # sigma_{i,0} = 0
    sent = [0] * N
    xs, sigmas = {}, {}
    for k in range(1, L + 1):
        # Step 1: generate, accumulate, transmit
        x = []
        for i in range(N):
            if k <= c:
                C[i] = C[i] + D[i][k - 1]
            x.append(C[i].copy())          # x_{i,k} leaves worker i
            sent[i] += p
        # Step 2: receive, store, update
        for i in range(N):
            C[i] = x[(i - 1) % N].copy()   # receive x_{i-1,k} into C_i
            if k <= N - 1:
                B[i][k - 1] = C[i].copy()
            else:
                j = k - N + 1
                C[i] = C[i] - D[i][j - 1]              # cancel delta_{i,j}
                if literal_store:
                    D[i][j - 1] = D[i][j - 1] + C[i]   # = x_{i-1,k} in exact arithmetic
                else:
                    D[i][j - 1] = x[(i - 1) % N].copy()
        if trace:
            xs[k] = [v.copy() for v in x]
            sigmas[k] = [v.copy() for v in C]
    Y = [np.stack(B[i] + D[i], axis=1) for i in range(N)]
    extra = {"x": xs, "sigma": sigmas} if trace else {}
    return Y, sent, extra


def decode(Y: np.ndarray, R: np.ndarray, scale: float = 1.0) -> np.ndarray:
    """G_hat_i = Y_i R_i (Sec. II-A, decoding), times an output scale.
    scale = 1 is the paper's approximate sum; scale = 1/N gives the mean."""
    return scale * (np.asarray(Y, np.float64) @ np.asarray(R, np.float64))


def allreduce(grads, U, R, scale: float = 1.0, *, literal_store: bool = False):
    """Whole pipeline for N workers: chunk, encode, L rounds, decode.

    grads : sequence of N length-d vectors; U[i] c x c; R[i] (L+1) x c.
    Returns dict with 'out' (N x d), 'Delta', 'Y', and the counters.
    """
    N = len(grads)
    c = np.asarray(U[0]).shape[0]
    d = np.asarray(grads[0]).shape[0]
    p = d // c
    G = [chunk_matrix(g, c) for g in grads]
    Delta = [encode(G[i], U[i]) for i in range(N)]
    Y, sent, _ = run_rounds(Delta, literal_store=literal_store)
    out = np.stack([unchunk(decode(Y[i], R[i], scale)) for i in range(N)])
    return {
        "out": out, "Delta": Delta, "Y": Y,
        "values_sent_per_worker": sent,
        "values_stored_per_worker": (c + N) * p,   # D_1..D_c, B_1..B_{N-1}, C
        "rounds": num_rounds(N, c),
    }


def exact_sum(grads) -> np.ndarray:
    """sum_j g_j in fp64: the quantity CERAR approximates (diagnostic only)."""
    return np.sum(np.stack([np.asarray(g, np.float64) for g in grads]), axis=0)


def rel_l2(a, b) -> float:
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a - b))


# ---------------------------------------------------------------- structure

def m_matrix(U, i: int) -> np.ndarray:
    """M_i(U), an Nc x (L+1) matrix whose r-th block row is
    [0_{c x (N-1-r)}  U_{i+r}  0_{c x r}]   (Sec. II-B, displayed equation
    after the rate formulas)."""
    N = len(U)
    c = np.asarray(U[0]).shape[0]
    L = num_rounds(N, c)
    M = np.zeros((N * c, L + 1), dtype=np.asarray(U[0]).dtype)
    for r in range(N):
        M[r * c:(r + 1) * c, N - 1 - r:N - 1 - r + c] = U[(i + r) % N]
    return M


def stacked_gradients(G, i: int) -> np.ndarray:
    """G^(i) = [G_i | G_{i+1} | ... | G_{i+N-1}] (indices mod N)."""
    N = len(G)
    return np.concatenate([G[(i + r) % N] for r in range(N)], axis=1)


def target(N: int, c: int) -> np.ndarray:
    """T = 1_N (x) I_c."""
    return np.kron(np.ones((N, 1)), np.eye(c))


def window(Ri: np.ndarray, s: int, c: int) -> np.ndarray:
    """W_s(R_i) = R_i[s : s+c-1, :] (rows numbered from 0)."""
    return Ri[s:s + c, :]


def phi(U, R) -> float:
    """Phi(U, R) = sum_i || M_i(U) R_i - T ||_F^2 (Eq. F_unreg)."""
    N = len(U)
    c = np.asarray(U[0]).shape[0]
    T = target(N, c)
    return float(sum(np.linalg.norm(m_matrix(U, i) @ R[i] - T, "fro") ** 2 for i in range(N)))


def kappa2(A: np.ndarray) -> float:
    s = np.linalg.svd(np.asarray(A, np.float64), compute_uv=False)
    return float(s[0] / s[-1]) if s[-1] > 0 else float("inf")


def rates(N: int, c: int):
    """(communication rate L/c = 1+(N-2)/c, storage rate 1+N/c)."""
    return (num_rounds(N, c) / c, 1.0 + N / c)
