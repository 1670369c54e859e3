"""Pins of the oracle's ternary absmean quantiser (paper Eq. 1-3, Figure 10) and of
the scale -> (mult, shift) conversion: the paper's closed form for the ternary
distribution at initialisation, hand-worked rows, ties, invariances, and exact
rational arithmetic."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_cost_shares.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if "=" in line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def test_he_normal_init_gives_the_papers_distribution(oracle):
    """Supplementary A.1: with W ~ N(0, 2/cout), about 31 % zeros and 34.5 % each of +-1."""
    g = golden()
    cout, cin = 384, 4096
    rng = np.random.default_rng(0)
    w = rng.normal(0.0, math.sqrt(2.0 / cout), size=(cout, cin)).astype(np.float32)
    q, alpha = oracle.quantize_ternary(w)
    n = q.size
    p0, pp, pm = (q == 0).sum() / n, (q == 1).sum() / n, (q == -1).sum() / n
    # the paper rounds to two / three digits; the exact value is erf(sqrt(1/pi)/2) = 0.3101
    assert abs(p0 - g["ternary_zero_fraction_init"]) < 0.005
    assert abs(pp - g["ternary_plus_fraction_init"]) < 0.005
    assert abs(pm - g["ternary_plus_fraction_init"]) < 0.005
    assert abs(p0 - math.erf(0.5 * math.sqrt(2.0 / math.pi) / math.sqrt(2.0))) < 4 * math.sqrt(0.31 * 0.69 / n)
    # alpha approximates E|W| = sigma * sqrt(2/pi) (Eq. 9-10 of the supplement)
    assert np.allclose(alpha, math.sqrt(2.0 / cout) * math.sqrt(2.0 / math.pi), rtol=0.05)


def test_hand_worked_rows(oracle):
    # row 0: |w| mean = 1 -> ratios equal the weights: 0.4 -> 0, 0.6 -> 1, -1.6 -> -2 -> -1, 1.4 -> 1
    # row 1: all equal -> ratio +-1 exactly
    # row 2: all zero -> mean clamped to eps, ratio 0
    w = np.array([[0.4, 0.6, -1.6, 1.4], [-3.0, 3.0, 3.0, -3.0], [0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    q, alpha = oracle.quantize_ternary(w)
    assert q.tolist() == [[0, 1, -1, 1], [-1, 1, 1, -1], [0, 0, 0, 0]]
    assert np.allclose(alpha, [1.0, 3.0, 0.0], atol=1e-7)


def test_ties_go_to_even(oracle):
    # mean |w| = 1 exactly (float32-exact values): ratios 0.5, -0.5, 1.5, -1.5, 2.5, 0, ...
    row = np.array([0.5, -0.5, 1.5, -1.5, 2.5, 0.0, 0.25, 1.25], dtype=np.float32)
    assert float(np.abs(row).mean()) == 1.0
    q, _ = oracle.quantize_ternary(row[None, :])
    assert q[0].tolist() == [0, 0, 1, -1, 1, 0, 0, 1]


def test_invariances(oracle):
    rng = np.random.default_rng(1)
    w = rng.normal(size=(37, 145)).astype(np.float32)
    q, alpha = oracle.quantize_ternary(w)
    q2, alpha2 = oracle.quantize_ternary(4.0 * w)          # exact scaling by a power of two
    assert np.array_equal(q, q2) and np.allclose(alpha2, 4.0 * alpha, rtol=1e-12)
    q3, _ = oracle.quantize_ternary(-w)
    assert np.array_equal(q3, -q)
    perm = rng.permutation(145)
    q4, alpha4 = oracle.quantize_ternary(w[:, perm])
    assert np.array_equal(q4, q[:, perm]) and np.allclose(alpha4, alpha, rtol=1e-12)
    # the decision itself, in exact arithmetic: |w| * cin versus half / three halves of sum |w|
    s = [sum(Fraction(float(abs(v))) for v in row) for row in w]
    for i in range(0, 37, 6):
        for j in range(0, 145, 7):
            ratio = Fraction(float(w[i, j])) * 145 / s[i]
            want = 0 if abs(ratio) < Fraction(1, 2) else (1 if ratio > 0 else -1)
            assert q[i, j] == want


def test_eps_guard_is_a_clamp_of_the_mean(oracle):
    """Figure 10 clamps the mean at eps; Eq. 3 adds eps.  With mean = 1e-6 < eps the ratio
    is w / 1e-5: 6e-6 -> 0.6 -> 1 under the clamp (adding eps would give 0.545 -> 1 too, so the
    row also holds 5.2e-6 -> 0.52 -> 1 against 0.473 -> 0)."""
    row = np.zeros(16, dtype=np.float32)
    row[0], row[1] = 6e-6, 5.2e-6
    row[2] = 16e-6 - row[0] - row[1]        # mean |w| = 1e-6
    q, alpha = oracle.quantize_ternary(row[None, :])
    assert abs(alpha[0] - 1e-6) < 1e-9
    assert q[0, 0] == 1 and q[0, 1] == 1


def test_requant_from_scale_exact(oracle):
    rng = np.random.default_rng(2)
    scales = list(2.0 ** rng.uniform(-31.9, -0.01, size=300)) + [0.5, 0.25, 2.0 ** -13, 0.75 * 2.0 ** -8,
                                                                  (1 - 2.0 ** -33) * 2.0 ** -9]
    for sc in scales:
        mult, shift = oracle.requant_from_scale(sc)
        assert (1 << 30) <= mult < (1 << 31) and 0 <= shift <= 31
        exact = Fraction(sc)
        got = Fraction(mult, 1 << (31 + shift))
        assert abs(got - exact) <= Fraction(1, 1 << (32 + shift))      # nearest multiple of 2^-(31+shift)
    assert oracle.requant_from_scale(0.5) == (1 << 30, 0)
    assert oracle.requant_from_scale(2.0 ** -13) == (1 << 30, 12)
    for bad in (0.0, -1.0, 1.0, 3.0, 2.0 ** -40):
        with pytest.raises(ValueError):
            oracle.requant_from_scale(bad)
