"""Pins of oracle/mixed.py (bfloat16 messages): the rounding against worked values, IEEE
properties and torch's own conversion (an independent implementation); the rounds against the
exact protocol where no rounding can occur, and against the error bound that 8-bit messages imply."""
import numpy as np
import pytest

from oracle import mixed as Mx
from oracle import protocol as P


def test_round_bf16_worked_values_and_ties_to_even():
    f = np.float32
    cases = [
        (1.0, 1.0), (-2.5, -2.5), (0.0, 0.0),
        (1.0 + 2.0 ** -8, 1.0),                       # tie, even mantissa below: down
        (1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -6),       # tie, odd mantissa below: up (to 1 + 4 * 2^-8)
        (1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 2.0 ** -7),   # just above the tie: up
        (1.0 + 2.0 ** -9, 1.0),                       # below half: down
        (3.0e38, 3.0041e38),                          # largest binade, no overflow
        (1.5 * 2.0 ** -130, 1.5 * 2.0 ** -130),       # subnormal, representable
    ]
    for x, want in cases:
        got = float(Mx.round_bf16(np.array([x], dtype=f))[0])
        assert got == pytest.approx(want, rel=2e-4) and float(f(got)) == got, (x, got, want)
    exact = [(1.0 + 2.0 ** -8, 1.0), (1.0 + 3 * 2.0 ** -8, 1.015625), (1.0 + 2.0 ** -9, 1.0), (-1.0 - 3 * 2.0 ** -8, -1.015625)]
    for x, want in exact:
        assert float(Mx.round_bf16(np.array([x], dtype=f))[0]) == want


def test_round_bf16_properties_and_agreement_with_torch():
    import torch
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(200000) * 10.0 ** rng.integers(-30, 30, 200000),
                        rng.integers(-1000, 1000, 5000).astype(np.float64) / 256.0]).astype(np.float32)
    r = Mx.round_bf16(x)
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)                       # 8 significant bits
    ok = np.isfinite(r)
    assert np.all(np.abs(r[ok].astype(np.float64) - x[ok]) <= 2.0 ** -8 * np.abs(x[ok].astype(np.float64)) * (1 + 1e-12) + 1e-45)
    assert np.array_equal(Mx.round_bf16(r), r)                             # idempotent
    assert np.array_equal(Mx.round_bf16(-x), -r)                           # symmetric
    order = np.argsort(x[ok])
    assert np.all(np.diff(r[ok][order]) >= 0)                              # monotone
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()   # torch's conversion is RNE too
    assert np.array_equal(t.view(np.uint32), r.view(np.uint32))


@pytest.mark.parametrize("N,c", [(2, 2), (3, 5), (4, 8), (5, 6)])
def test_rounds_equal_the_exact_protocol_when_nothing_rounds(N, c):
    """Small integers: every partial sum of at most N of them is a bfloat16 number, so the rounded
    protocol must give exactly what Algorithm 1 gives (indices, order of cancel and add, landing slots)."""
    rng = np.random.default_rng(N * 10 + c)
    p = 7
    Delta = [rng.integers(-7, 8, (p, c)).astype(np.float64) for _ in range(N)]
    Y_exact, _, _ = P.run_rounds(Delta)
    Y = Mx.run_rounds_bf16([d.astype(np.float32) for d in Delta])
    for i in range(N):
        assert Y[i].dtype == np.float32 and np.array_equal(Y[i].astype(np.float64), Y_exact[i])


def test_rounds_error_stays_within_what_the_message_precision_implies():
    """Every message carries a relative rounding error of at most 2^-8 and a message is a sum of at
    most N encoded vectors that is rounded at every hop: |Y - Y_exact| <= N * 2^-8 * max|partial sum|
    (crude), and the error is not zero for generic data (the rounding is really applied)."""
    rng = np.random.default_rng(3)
    N, c, p = 4, 9, 64
    Delta = [rng.standard_normal((p, c)) for _ in range(N)]
    Y_exact, _, _ = P.run_rounds(Delta)
    Y = Mx.run_rounds_bf16([d.astype(np.float32) for d in Delta])
    worst = 0.0
    for i in range(N):
        err = np.abs(Y[i].astype(np.float64) - Y_exact[i])
        # the last column is delta_c itself, never transmitted
        assert np.array_equal(Y[i][:, -1], Delta[i][:, -1].astype(np.float32))
        worst = max(worst, err[:, :-1].max())
        assert np.all((Y[i][:, :-1].view(np.uint32) & 0xFFFF) == 0)      # what was received is bfloat16
    bound = N * 2.0 ** -8 * N * np.abs(np.stack(Delta)).max() * 1.01
    assert 1e-4 < worst <= bound
    assert Mx.message_bytes(N, c, p) * 2 == 4 * p * P.num_rounds(N, c)


# ---------------------------------------------------------------- 8-bit messages

def test_round_e4m3_worked_values():
    """Values worked out by hand from the format (3 mantissa bits, bias 7, subnormal step 2^-9, max 448)."""
    cases = [
        (0.1, 0.1015625, 0b0_0011_101),       # 1.6 * 2^-4 -> 1.625 * 2^-4
        (17.0, 16.0, 0b0_1011_000),           # tie between 16 and 18: even mantissa (000)
        (19.0, 20.0, 0b0_1011_010),           # tie between 18 (001) and 20 (010): even
        (2.0 ** -10, 0.0, 0),                 # tie between 0 and the smallest subnormal: even (0)
        (3 * 2.0 ** -10, 2.0 ** -8, 2),       # tie between 1 and 2 subnormal steps: even (2)
        (2.0 ** -6, 2.0 ** -6, 0b0_0001_000),  # smallest normal
        (448.0, 448.0, 0b0_1111_110), (1.0e4, 448.0, 0b0_1111_110),        # largest finite; clamped beyond
        (-0.3, -0.3125, 0b1_0101_010), (1.0, 1.0, 0b0_0111_000), (0.0, 0.0, 0),
    ]
    for x, want, code in cases:
        v, cd = Mx.round_e4m3(np.array([x], dtype=np.float32))
        assert float(v[0]) == want and int(cd[0]) == code, (x, float(v[0]), int(cd[0]))


def test_round_e4m3_properties_and_agreement_with_torch():
    import torch
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(300000) * np.exp(rng.uniform(-9, 5.5, 300000))).astype(np.float32)
    x = np.clip(x, -448, 448)
    v, code = Mx.round_e4m3(x)
    t = torch.from_numpy(x).to(torch.float8_e4m3fn)                        # an independent implementation
    assert np.array_equal(t.view(torch.uint8).numpy(), code)
    assert np.array_equal(t.to(torch.float32).numpy(), v)
    big = np.abs(x) >= 2.0 ** -6
    assert np.all(np.abs(v[big].astype(np.float64) - x[big]) <= 2.0 ** -4 * np.abs(x[big].astype(np.float64)))
    assert np.all(np.abs(v[~big].astype(np.float64) - x[~big]) <= 2.0 ** -10)      # half a subnormal step
    assert np.array_equal(Mx.round_e4m3(v)[0], v)                          # idempotent
    assert np.array_equal(Mx.round_e4m3(-x)[0], -v)
    order = np.argsort(x)
    assert np.all(np.diff(v[order]) >= 0)
    assert len(np.unique(code)) > 200                                      # the whole code space is in use


def test_tile_scales_use_the_range_without_clamping():
    rng = np.random.default_rng(2)
    tile = 64
    x = (rng.standard_normal(10 * tile + 17) * np.repeat(10.0 ** rng.uniform(-12, 12, 11), tile)[:10 * tile + 17]).astype(np.float32)
    x[3 * tile:4 * tile] = 0.0                                             # a tile of zeros
    x[5 * tile] = 448.0 * 2.0 ** 3                                         # amax exactly 448 * 2^3: e = 3, not 4
    x[5 * tile + 1:6 * tile] *= 1e-12
    e = Mx.tile_scale_exponents(x, tile)
    assert e[3] == 0 and e[5] == 3
    for t in range(len(e)):
        amax = np.abs(x[t * tile:(t + 1) * tile]).max()
        if amax > 0:
            assert amax * 2.0 ** -float(e[t]) <= 448.0 and amax * 2.0 ** -float(e[t] - 1) > 448.0
    codes, scales, back = Mx.quantize_fp8_tiles(x, tile)
    assert codes.dtype == np.uint8 and codes.shape == x.shape and scales.shape == e.shape
    assert np.array_equal(scales, (2.0 ** e.astype(np.float64)).astype(np.float32))
    amax_pos = np.repeat([np.abs(x[t * tile:(t + 1) * tile]).max() for t in range(len(e))], tile)[:x.size]
    # error per element: half a spacing of the scaled value, i.e. at most 2^-4 of the tile's largest magnitude
    assert np.all(np.abs(back.astype(np.float64) - x) <= 2.0 ** -4 * amax_pos * (1 + 1e-12))
    assert np.any(back != x)
    # a decoder that only has codes and scales reconstructs the same values (torch's table as the decoder)
    import torch
    dec = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy() * np.repeat(scales, tile)[:x.size]
    assert np.array_equal(dec, back)


@pytest.mark.parametrize("N,c", [(2, 2), (3, 5), (4, 8)])
def test_fp8_rounds_equal_the_exact_protocol_when_nothing_rounds(N, c):
    """Small integers (|sum of N of them| <= 14 < 16, where e4m3 still holds every integer, and every
    tile's scale is a power of two): the 8-bit protocol must reproduce the exact one."""
    rng = np.random.default_rng(N * 10 + c)
    p = 37
    top = 14 // N
    Delta = [rng.integers(-top, top + 1, (p, c)).astype(np.float64) for _ in range(N)]
    Y_exact, _, _ = P.run_rounds(Delta)
    Y = Mx.run_rounds_fp8([d.astype(np.float32) for d in Delta], tile=16)
    for i in range(N):
        assert np.array_equal(Y[i].astype(np.float64), Y_exact[i])


def test_fp8_rounds_error_and_bytes():
    rng = np.random.default_rng(4)
    N, c, p, tile = 4, 9, 256, 64
    Delta = [rng.standard_normal((p, c)) for _ in range(N)]
    Y_exact, _, _ = P.run_rounds(Delta)
    Y = Mx.run_rounds_fp8([d.astype(np.float32) for d in Delta], tile)
    worst = 0.0
    for i in range(N):
        err = np.abs(Y[i].astype(np.float64) - Y_exact[i])
        assert np.array_equal(Y[i][:, -1], Delta[i][:, -1].astype(np.float32))    # delta_c never travels
        worst = max(worst, err[:, :-1].max())
    bound = N * 2.0 ** -4 * N * np.abs(np.stack(Delta)).max() * 1.01
    assert 1e-2 < worst <= bound
    assert Mx.message_bytes_fp8(N, c, p, tile) == (p + 4 * (p // tile)) * P.num_rounds(N, c)
