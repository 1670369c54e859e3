"""Pins of the oracle's per-sample absmax activation quantiser (paper Eq. 6-7 and the
activation figure of the pseudocode appendix): hand-worked samples, ties, what the definition
fixes for any input (the largest element maps to +-127, scale and sign symmetries, one scale per
sample), the decision redone in exact rational arithmetic, and the degenerate samples."""
from fractions import Fraction

import numpy as np
import pytest


def test_hand_worked_samples(oracle):
    # sample 0: max |x| = 127 -> scale 1: values round to themselves, 0.5 -> 0, 1.5 -> 2, 2.5 -> 2
    # sample 1: max |x| = 2 -> scale 63.5: 1 -> 63.5 -> 64 (tie to even), -2 -> -127, 0.1 -> 6.35 -> 6
    x = np.array([[127.0, 0.5, 1.5, 2.5, -126.5, -0.4], [1.0, -2.0, 0.1, 0.0, 2.0, -1.0]], dtype=np.float32)
    q, gamma, scale = oracle.quantize_act_absmax(x)
    assert gamma.tolist() == [127.0, 2.0]
    assert scale.tolist() == [1.0, 63.5]
    assert q[0].tolist() == [127, 0, 2, 2, -126, 0]
    assert q[1].tolist() == [64, -127, 6, 0, 127, -64]


def test_largest_element_maps_to_127_and_codes_stay_in_range(oracle):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((6, 7, 5, 9)) * rng.uniform(1e-3, 1e3, size=(6, 1, 1, 1))).astype(np.float32)
    q, gamma, scale = oracle.quantize_act_absmax(x)
    flat, qf = x.reshape(6, -1), q.reshape(6, -1)
    for i in range(6):
        j = int(np.argmax(np.abs(flat[i])))
        assert gamma[i] == np.abs(flat[i]).max()
        assert abs(int(qf[i, j])) == 127 and np.sign(qf[i, j]) == np.sign(flat[i, j])
        assert qf[i].min() >= -127 and qf[i].max() <= 127      # -128 is unreachable: |x| <= gamma
        # monotone: a larger value never gets a smaller code
        order = np.argsort(flat[i], kind="stable")
        assert np.all(np.diff(qf[i][order].astype(np.int32)) >= 0)


def test_decision_in_exact_rationals(oracle):
    """Away from ties the code is round(x * 127 / gamma) as a real number: the two binary32
    roundings cannot move the product by more than 2^-22 of its size."""
    rng = np.random.default_rng(6)
    x = rng.uniform(-3.0, 3.0, size=(4, 500)).astype(np.float32)
    q, gamma, _ = oracle.quantize_act_absmax(x)
    checked = 0
    for i in range(4):
        g = Fraction(float(gamma[i]))
        for j in range(500):
            v = Fraction(float(x[i, j])) * 127 / g
            frac = v - (v.numerator // v.denominator)
            if abs(frac - Fraction(1, 2)) < Fraction(1, 1000):
                continue                                        # too close to a tie to call
            want = (v + Fraction(1, 2)).numerator // (v + Fraction(1, 2)).denominator
            assert int(q[i, j]) == want, (i, j, float(v))
            checked += 1
    assert checked > 1900


def test_scale_and_sign_symmetries(oracle):
    rng = np.random.default_rng(7)
    x = rng.standard_normal((3, 64)).astype(np.float32)
    q, gamma, scale = oracle.quantize_act_absmax(x)
    # a power of two times the input: same codes, gamma scaled, scale divided (all exact in binary32)
    q2, gamma2, scale2 = oracle.quantize_act_absmax(x * np.float32(8.0))
    assert np.array_equal(q, q2) and np.array_equal(gamma2, gamma * 8) and np.array_equal(scale2, scale / 8)
    # negation: codes negate (ties to even is symmetric)
    qn, gamman, _ = oracle.quantize_act_absmax(-x)
    assert np.array_equal(qn.astype(np.int32), -q.astype(np.int32)) and np.array_equal(gamman, gamma)
    # samples do not see each other: quantising one sample alone gives the same codes
    for i in range(3):
        qi, _, _ = oracle.quantize_act_absmax(x[i:i + 1])
        assert np.array_equal(qi[0], q[i])
    # a permutation inside a sample permutes the codes
    perm = rng.permutation(64)
    qp, _, _ = oracle.quantize_act_absmax(x[:, perm])
    assert np.array_equal(qp, q[:, perm])


def test_zero_and_tiny_samples(oracle):
    """An all-zero sample has gamma 0: the figure clamps the divisor to eps, every code is 0.
    A sample below eps is scaled by 127/eps and does not reach 127."""
    x = np.zeros((2, 16), dtype=np.float32)
    x[1, 3] = 5e-6
    q, gamma, scale = oracle.quantize_act_absmax(x)
    assert gamma.tolist() == [0.0, np.float32(5e-6)]
    assert scale[0] == np.float32(127.0) / np.float32(1e-5) and scale[1] == scale[0]
    assert not q[0].any()
    assert q[1, 3] == 64 and q[1].astype(np.int32).sum() == 64           # 5e-6 * 1.27e7 = 63.5 -> 64


def test_already_integer_inputs_survive(oracle):
    """int8-valued activations whose largest magnitude is 127 come back unchanged: the
    special case in which the quantiser is the identity."""
    rng = np.random.default_rng(8)
    xi = rng.integers(-127, 128, size=(2, 300)).astype(np.float32)
    xi[:, 0] = 127.0
    q, _, scale = oracle.quantize_act_absmax(xi)
    assert scale.tolist() == [1.0, 1.0]
    assert np.array_equal(q.astype(np.float32), xi)
