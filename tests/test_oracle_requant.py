"""Pins for the fixed-point requantiser: exact rational arithmetic, float64
closed form, hand-built ties, symmetry."""
from fractions import Fraction
import math

import numpy as np


def exact(t, mult, shift, lo, hi):
    """round-half-away of t*mult / 2^(31+shift) in rational arithmetic."""
    v = Fraction(t * mult, 1 << (31 + shift))
    a = abs(v)
    q = math.floor(a + Fraction(1, 2))
    q = q if v >= 0 else -q
    return min(hi, max(lo, q))


def test_against_exact_rationals(oracle):
    rng = np.random.default_rng(0)
    for _ in range(300):
        mult = int(rng.integers(1 << 30, 1 << 31))
        shift = int(rng.integers(0, 32))
        ts = rng.integers(-(1 << 18), 1 << 18, size=64)
        for t in ts.tolist() + [0, 1, -1, (1 << 18), -(1 << 18), 2**31 - 1, -2**31]:
            assert oracle.requant_scalar(t, mult, shift, -128, 127) == exact(t, mult, shift, -128, 127)


def test_extreme_constants(oracle):
    for mult in (0, 1, 1 << 30, (1 << 31) - 1):
        for shift in (0, 8, 12, 31):
            for t in (-300000, -1, 0, 1, 255, 256, 300000):
                for lo, hi in ((0, 127), (-128, 127), (-5, 5)):
                    assert oracle.requant_scalar(t, mult, shift, lo, hi) == exact(t, mult, shift, lo, hi)


def test_float64_closed_form(oracle):
    # |p| < 2^49 so p / 2^s is exact in binary64
    rng = np.random.default_rng(1)
    t = rng.integers(-(1 << 17), 1 << 17, size=20000).astype(np.int32)
    for mult, shift in [(1 << 30, 8), ((1 << 31) - 1, 12), (1518500250, 10)]:
        v = t.astype(np.float64) * float(mult) / float(2 ** (31 + shift))
        want = np.copysign(np.floor(np.abs(v) + 0.5), v)
        want = np.clip(want, -128, 127).astype(np.int32)
        got = oracle.requant(t, mult, shift, -128, 127)
        assert np.array_equal(got, want)


def test_ties_round_away_from_zero(oracle):
    # mult = 2^30: scale = 2^-(shift+1); t an odd multiple of 2^shift is a tie
    for shift in (0, 3, 8, 12):
        for k in (1, 3, 5, 77):
            t = k * (1 << shift)
            q = oracle.requant_scalar(t, 1 << 30, shift, -128, 127)
            assert q == (k + 1) // 2
            qn = oracle.requant_scalar(-t, 1 << 30, shift, -128, 127)
            assert qn == -((k + 1) // 2)
    # one step below a tie rounds down in magnitude
    assert oracle.requant_scalar(3 * 256 - 1, 1 << 30, 8, -128, 127) == 1
    assert oracle.requant_scalar(-(3 * 256 - 1), 1 << 30, 8, -128, 127) == -1


def test_odd_symmetry_and_monotonicity(oracle):
    rng = np.random.default_rng(2)
    t = np.arange(-70000, 70000, dtype=np.int32)
    for _ in range(10):
        mult = int(rng.integers(1 << 30, 1 << 31))
        shift = int(rng.integers(8, 13))
        q = oracle.requant(t, mult, shift, -127, 127)
        qn = oracle.requant(-t, mult, shift, -127, 127)
        assert np.array_equal(q, -qn)
        assert (np.diff(q) >= 0).all()


def test_clamp(oracle):
    assert oracle.requant_scalar(10**6, (1 << 31) - 1, 8, 0, 127) == 127
    assert oracle.requant_scalar(-10**6, (1 << 31) - 1, 8, 0, 127) == 0
    assert oracle.requant_scalar(-10**6, (1 << 31) - 1, 8, -128, 127) == -128
    assert oracle.requant_scalar(700, 1 << 30, 0, 3, 9) == 9
    assert oracle.requant_scalar(2, 1 << 30, 0, 3, 9) == 3
