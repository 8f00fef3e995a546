"""CERAR data path in plain numpy fp64, written from the paper's definitions.

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
    """The L ring rounds for all N workers, evaluated from the update equations
    (Eq. update_eqns):

        x_{i,k}     = delta_{i,k} + sigma_{i,k-1}        for 1 <= k <= c,
                    = sigma_{i,k-1}                      for c < k <= L,
        sigma_{i,k} = x_{i-1,k}                          for 1 <= k <= N-1,
                    = x_{i-1,k} - delta_{i,k-N+1}        for N <= k <= L,

    with sigma_{i,0} = 0 and worker indices modulo N.  Worker i observes
    y_{i,k} = x_{i-1,k} in round k (k = 1..L) and keeps y_{i,L+1} = delta_{i,c},
    which no round overwrites; Y_i = [y_{i,1} .. y_{i,L+1}] is the order in which
    Sec. II lists the stored observations (the N-1 dedicated buffers first, then
    the c slots that held the encoded vectors).

    Delta : list of N arrays (p x c); column j-1 is delta_{i,j}.
    literal_store : evaluate the same rounds on the storage slots D, B, C of
        Sec. II instead (storage_rounds below), where a received vector reaches
        its slot as "old content plus the new state".  Equal up to rounding.
    trace : also return the messages x[k][i] and the states sigma[k][i].

    Returns (Y, sent, extra): Y[i] is the p x (L+1) observation matrix, sent[i]
    the number of real values worker i transmitted, extra the trace (or empty).
    """
    if literal_store:
        return storage_rounds(Delta, trace=trace)
    N = len(Delta)
    p, c = Delta[0].shape
    L = num_rounds(N, c)

    def delta(i, j):                       # delta_{i,j}, j = 1..c
        return np.asarray(Delta[i % N][:, j - 1], dtype=np.float64)

    sigma = [np.zeros(p, dtype=np.float64) for _ in range(N)]     # sigma_{i,0}
    observed = [[] for _ in range(N)]
    xs, sigmas = {}, {}
    for k in range(1, L + 1):
        x = [delta(i, k) + sigma[i] if k <= c else sigma[i].copy() for i in range(N)]
        nxt = []
        for i in range(N):
            y = x[(i - 1) % N]
            observed[i].append(y.copy())
            nxt.append(y.copy() if k <= N - 1 else y - delta(i, k - N + 1))
        sigma = nxt
        if trace:
            xs[k] = [v.copy() for v in x]
            sigmas[k] = [v.copy() for v in sigma]
    Y = [np.stack(observed[i] + [delta(i, c).copy()], axis=1) for i in range(N)]
    sent = [L * p] * N                     # one length-p message per worker and round
    extra = {"x": xs, "sigma": sigmas} if trace else {}
    return Y, sent, extra


def storage_rounds(Delta, *, trace: bool = False):
    """The same rounds carried out on the storage of Sec. II: per worker the slots
    D_1..D_c (initially the encoded vectors), the dedicated buffers B_1..B_{N-1}
    and the rolling buffer C (initially zero).  What is sent in round k is the
    content of C after D_k was added to it (k <= c); what arrives replaces C, is
    copied to B_k while k <= N-1, and from round N on the returning delta in
    D_{k-N+1} is taken out of C and the slot then receives "its old content plus
    C", which is the arrived vector in exact arithmetic.  Kept as a check of
    run_rounds (the two must agree to rounding) and of the storage count."""
    N = len(Delta)
    p, c = Delta[0].shape
    L = num_rounds(N, c)
    D = [[np.array(Delta[i][:, j], dtype=np.float64) for j in range(c)] for i in range(N)]
    B = [[None] * (N - 1) for _ in range(N)]
    C = [np.zeros(p, dtype=np.float64) for _ in range(N)]
    sent = [0] * N
    xs, sigmas = {}, {}
    for k in range(1, L + 1):
        for i in range(N):
            if k <= c:
                C[i] = C[i] + D[i][k - 1]
        outgoing = [C[i].copy() for i in range(N)]
        for i in range(N):
            sent[i] += p
            C[i] = outgoing[(i - 1) % N].copy()
            if k <= N - 1:
                B[i][k - 1] = C[i].copy()
            else:
                slot = k - N            # 0-based index of D_{k-N+1}
                C[i] = C[i] - D[i][slot]
                D[i][slot] = D[i][slot] + C[i]
        if trace:
            xs[k] = outgoing
            sigmas[k] = [v.copy() for v in C]
    Y = [np.stack(B[i] + D[i], axis=1) for i in range(N)]
    return Y, sent, ({"x": xs, "sigma": sigmas} if trace else {})


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
