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
