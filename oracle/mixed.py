"""Ring rounds of CERAR with low-precision messages (bfloat16 transport).

Test infrastructure only (see the package docstring).  The paper leaves the combination
with gradient quantisation open (Sec. I, Related Work, only notes that compression is
complementary to the coding and could be combined with it).  This module states one such
combination so that the device path has something to be compared with: Algorithm 1 (Sec. II)
unchanged, except that every transmitted message x_{i,k} is rounded to bfloat16 by its sender;
the receiver stores and uses the rounded vector.

A rounding is a decision, and both sides must take it in the same precision (the device's):
the workers' arithmetic here is IEEE binary32 (one rounding per sum or difference of the update
equations, the message rounded once more by its sender), on binary32 encoded vectors that are
an INPUT (seeded synthetic ones, or an fp64 encode cast to binary32).  Given the same Delta the
observations Y are therefore fixed bit for bit.
"""
from __future__ import annotations

import numpy as np

from . import protocol


def round_bf16(x) -> np.ndarray:
    """binary32 -> bfloat16 (8 significant bits), round to nearest, ties to even, returned
    as binary32.  Written on the bit pattern: keep the upper 16 bits, round on the lower 16."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    lower = bits & 0xFFFF
    upper = bits >> 16
    up = (lower > 0x8000) | ((lower == 0x8000) & ((upper & 1) == 1))
    out = ((upper + up.astype(np.uint64)) << 16).astype(np.uint32)
    res = out.view(np.float32).copy()
    nan = np.isnan(x)
    res[nan] = np.float32(np.nan)
    return res.reshape(x.shape)


def run_rounds_bf16(Delta32):
    """The L rounds for all N workers with binary32 worker arithmetic and bfloat16 messages:
    the update equations (Eq. update_eqns) with one rounding added where a vector leaves its sender,

        x_{i,k}     = bf16( delta_{i,k} + sigma_{i,k-1} )   (k <= c),   bf16( sigma_{i,k-1} )   (k > c),
        sigma_{i,k} = x_{i-1,k}   (k <= N-1),   x_{i-1,k} - delta_{i,k-N+1}   (k >= N),

    every sum and difference rounded to binary32.  The receiver keeps the rounded vector as
    its observation y_{i,k}; y_{i,L+1} = delta_{i,c} never travels and stays binary32.

    Delta32 : list of N arrays (p x c), binary32; column j-1 is delta_{i,j}.
    Returns Y: list of N arrays (p x (L+1)), binary32, columns y_{i,1} .. y_{i,L+1}.
    """
    N = len(Delta32)
    p, c = Delta32[0].shape
    L = protocol.num_rounds(N, c)
    f32 = np.float32

    def delta(i, j):
        return np.asarray(Delta32[i % N][:, j - 1], dtype=f32)

    sigma = [np.zeros(p, dtype=f32) for _ in range(N)]
    observed = [[] for _ in range(N)]
    for k in range(1, L + 1):
        x = [round_bf16((delta(i, k) + sigma[i]).astype(f32) if k <= c else sigma[i]) for i in range(N)]
        nxt = []
        for i in range(N):
            y = x[(i - 1) % N]
            observed[i].append(y.copy())
            nxt.append(y.copy() if k <= N - 1 else (y - delta(i, k - N + 1)).astype(f32))
        sigma = nxt
    return [np.stack(observed[i] + [delta(i, c).copy()], axis=1).astype(f32) for i in range(N)]


def message_bytes(N: int, c: int, p: int) -> int:
    """Bytes one worker forwards over the L rounds with 2-byte messages."""
    return 2 * p * protocol.num_rounds(N, c)
