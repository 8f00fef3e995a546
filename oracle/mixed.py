"""Ring rounds of CERAR with low-precision messages (bfloat16, and 8-bit e4m3 with a scale per tile).

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


# ---------------------------------------------------------------- 8-bit messages (e4m3, scale per tile)

E4M3_MAX = 448.0            # largest finite value of the 8-bit format with 4 exponent and 3 mantissa bits
FP8_TILE = 1024             # positions that share one power-of-two scale


def round_e4m3(x):
    """binary32 -> the nearest value of the 8-bit floating-point format e4m3 ("fn" variant: exponent
    bias 7, no infinities, largest finite value 448, subnormals in steps of 2^-9), round to nearest,
    ties to even, values beyond 448 clamped to +-448.  Returns (values as binary32, codes as uint8:
    sign << 7 | exponent field << 3 | mantissa field).  Written from the format's definition: the
    spacing of representable values around x is 2^(max(floor(log2 |x|), -6) - 3)."""
    x = np.ascontiguousarray(x, dtype=np.float32).astype(np.float64)
    a = np.abs(x)
    _, e = np.frexp(a)                                   # a = m 2^e with m in [0.5, 1): floor(log2 a) = e - 1
    q = np.maximum(e - 1, -6) - 3                        # exponent of the spacing
    y = np.rint(np.ldexp(a, -q))                         # numpy rounds halves to even
    y = np.minimum(np.ldexp(y, q), E4M3_MAX)
    # codes
    _, e2 = np.frexp(y)
    fe = e2 - 1
    normal = y >= 2.0 ** -6
    E = np.where(normal, fe + 7, 0).astype(np.int64)
    M = np.where(normal, np.rint((np.ldexp(y, -np.where(normal, fe, 0)) - 1.0) * 8.0), np.rint(np.ldexp(y, 9))).astype(np.int64)
    code = ((np.signbit(x).astype(np.int64) << 7) | (E << 3) | M).astype(np.uint8)
    return np.copysign(y, x).astype(np.float32), code


def tile_scale_exponents(x, tile: int = FP8_TILE):
    """Per tile of `tile` consecutive positions the smallest integer e with max|x| 2^-e <= 448 (so that
    the scaled tile fits the format without clamping), 0 for a tile of zeros, kept within [-100, 100] so
    that 2^e and the scaled values stay normal binary32 numbers.  x: length-p binary32 vector."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    p = x.shape[0]
    nt = (p + tile - 1) // tile
    e = np.zeros(nt, dtype=np.int64)
    for t in range(nt):
        amax = float(np.max(np.abs(x[t * tile:(t + 1) * tile])))
        if amax > 0.0 and np.isfinite(amax):
            m, E = np.frexp(amax)                        # amax = m 2^E, m in [0.5, 1); 448 = 0.875 * 2^9
            e[t] = E - 9 if m <= 0.875 else E - 8
    return np.clip(e, -100, 100)


def quantize_fp8_tiles(x, tile: int = FP8_TILE):
    """What the sender puts on the wire for one message: per tile a power-of-two scale 2^e (binary32)
    and per position the e4m3 code of x 2^-e.  Returns (codes uint8 [p], scales float32 [tiles],
    the values the receiver reconstructs, binary32 [p])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    p = x.shape[0]
    e = tile_scale_exponents(x, tile)
    e_pos = np.repeat(e, tile)[:p]
    scaled = np.ldexp(x.astype(np.float64), -e_pos).astype(np.float32)       # exact: a power of two
    vals, codes = round_e4m3(scaled)
    back = np.ldexp(vals.astype(np.float64), e_pos).astype(np.float32)
    return codes, np.ldexp(1.0, e).astype(np.float32), back


def run_rounds_fp8(Delta32, tile: int = FP8_TILE):
    """The L rounds with binary32 worker arithmetic and 8-bit messages: as run_rounds_bf16, with the
    sender's rounding replaced by quantize_fp8_tiles (scale per tile of positions, e4m3 codes)."""
    N = len(Delta32)
    p, c = Delta32[0].shape
    L = protocol.num_rounds(N, c)
    f32 = np.float32

    def delta(i, j):
        return np.asarray(Delta32[i % N][:, j - 1], dtype=f32)

    sigma = [np.zeros(p, dtype=f32) for _ in range(N)]
    observed = [[] for _ in range(N)]
    for k in range(1, L + 1):
        x = [quantize_fp8_tiles((delta(i, k) + sigma[i]).astype(f32) if k <= c else sigma[i], tile)[2] for i in range(N)]
        nxt = []
        for i in range(N):
            y = x[(i - 1) % N]
            observed[i].append(y.copy())
            nxt.append(y.copy() if k <= N - 1 else (y - delta(i, k - N + 1)).astype(f32))
        sigma = nxt
    return [np.stack(observed[i] + [delta(i, c).copy()], axis=1).astype(f32) for i in range(N)]


def message_bytes_fp8(N: int, c: int, p: int, tile: int = FP8_TILE) -> int:
    """Bytes one worker forwards over the L rounds with 1-byte codes and one 4-byte scale per tile."""
    return (p + 4 * ((p + tile - 1) // tile)) * protocol.num_rounds(N, c)
