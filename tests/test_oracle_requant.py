"""Pins of the oracle's per-token INT4 re-quantisation against what the definition and the
mathematics fix: hand-worked values, exact rational arithmetic, invariants."""
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

import oracle

GOLDEN = Path(__file__).parent / "golden" / "requant_small.txt"


def _cases():
    cur = {}
    for line in GOLDEN.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        cur[key] = rest.split()
        if key == "q":
            yield (np.array([float(v) for v in cur["y"]], dtype=np.float64), int(cur["s"][0], 16),
                   int(cur["inv"][0], 16), np.array([int(v) for v in cur["q"]], dtype=np.int8))
            cur = {}


def test_hand_worked_cases():
    n = 0
    for y, s_bits, inv_bits, q_exp in _cases():
        y16 = y.astype(np.float16)
        assert np.array_equal(y16.astype(np.float64), y), "fixture value not exact in fp16"
        q, s = oracle.requant_int4(y16[None, :])
        assert int(s.view(np.uint16)[0]) == s_bits
        assert int(oracle.requant_inverse(oracle.absmax_f16(y16[None, :])).view(np.uint16)[0]) == inv_bits
        assert np.array_equal(q[0], q_exp)
        n += 1
    assert n == 6


def _round_half_even(fr: Fraction) -> int:
    fl = fr.numerator // fr.denominator
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def _fp16_nearest(fr: Fraction) -> np.float16:
    """Round a positive rational to the nearest fp16, ties to even, by searching its neighbours."""
    lo = np.float16(float(fr))           # double rounding cannot cross more than one neighbour
    cands = {lo, np.nextafter(lo, np.float16(np.inf)), np.nextafter(lo, np.float16(0))}
    best = None
    for c in cands:
        d = abs(Fraction(float(c)) - fr)
        even = (int(np.float16(c).view(np.uint16)) & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, np.float16(c))
    return best[1]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_against_exact_rational_arithmetic(seed):
    """Scale and reciprocal are the correctly rounded fp16 quotients, and every code is the
    round-half-even of the exact rational product y * inv."""
    rng = np.random.default_rng(seed)
    scale = [1.0, 37.5, 2.0 ** -9][seed]
    y16 = (rng.standard_normal((6, 97)) * scale).astype(np.float16)
    y16[0, :8] = np.float16(scale) * np.array([0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, 7], np.float16)
    q, s = oracle.requant_int4(y16)
    inv = oracle.requant_inverse(oracle.absmax_f16(y16))
    for n in range(y16.shape[0]):
        amax = max(abs(Fraction(float(v))) for v in y16[n])
        assert s[n] == _fp16_nearest(amax / 7)
        inv_exact = _fp16_nearest(Fraction(7) / amax)
        assert np.isfinite(inv_exact) and inv[n] == inv_exact
        for m in range(y16.shape[1]):
            r = _round_half_even(Fraction(float(y16[n, m])) * Fraction(float(inv_exact)))
            assert q[n, m] == min(7, max(-8, r)), (n, m)


def test_invariants():
    rng = np.random.default_rng(7)
    y16 = (rng.standard_normal((16, 512)) * 3).astype(np.float16)
    q, s = oracle.requant_int4(y16)
    sf = s.astype(np.float64)[:, None]
    # the extreme element lands on +-7, nothing reaches -8 in the normal range
    idx = np.abs(y16.astype(np.float64)).argmax(axis=1)
    assert np.all(np.abs(q[np.arange(16), idx]) == 7) and q.min() >= -7 and q.max() <= 7
    # reconstruction error at most half a step (s * inv = 1 within two fp16 roundings)
    assert np.all(np.abs(q * sf - y16.astype(np.float64)) <= 0.5 * sf * (1 + 32 * 2.0 ** -11))
    # odd symmetry, and exact covariance under a power-of-two scaling
    qn, sn = oracle.requant_int4(-y16)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)
    q4, s4 = oracle.requant_int4((y16.astype(np.float32) * 4).astype(np.float16))
    assert np.array_equal(q4, q) and np.array_equal(s4.astype(np.float32), s.astype(np.float32) * 4)
    # a supplied absmax over a column range is the one that sets the step
    a = oracle.absmax_f16(y16, 100, 200)
    assert np.array_equal(a, np.abs(y16[:, 100:200]).max(axis=1))
    q2, s2 = oracle.requant_int4(y16[:, 100:200], a)
    q3, s3 = oracle.requant_int4(y16[:, 100:200])
    assert np.array_equal(q2, q3) and np.array_equal(s2, s3)
    assert np.array_equal(oracle.absmax_f16(y16, 5, 5), np.zeros(16, np.float16))
