"""Pins of the oracle's dynamic pointwise layer (pseudocode appendix, inference branch of the
quantised convolution module + the activation quantiser; Eq. 6-7): agreement of the dequantised
output with the real-number convolution of the dequantised operands, a hand-worked case, the
identity special case in exact rationals, what a change of alpha or of the input scale may and
may not change, and sample independence."""
from fractions import Fraction

import numpy as np
import pytest


def _case(seed, batch, rows, cin, cout):
    rng = np.random.default_rng(seed)
    x = rng.integers(-127, 128, size=(batch * rows, cin)).astype(np.int8)
    w = rng.integers(-1, 2, size=(cout, cin)).astype(np.int8)
    alpha = rng.uniform(0.01, 0.2, size=cout).astype(np.float32)
    gamma_x = rng.uniform(0.5, 8.0, size=batch).astype(np.float32)
    return x, w, alpha, gamma_x


def test_hand_worked(oracle):
    # one sample, two rows, cin 3, cout 2; gamma_x = 127 -> dq = 1; alpha = (0.5, 2)
    x = np.array([[10, -20, 30], [1, 2, 3]], dtype=np.int8)
    w = np.array([[1, 0, -1], [1, 1, 1]], dtype=np.int8)
    q, gy, sy, y = oracle.conv_dyn(x, w, np.array([0.5, 2.0], np.float32), np.array([127.0], np.float32), 2)
    # acc = [[-20, 20], [-2, 6]] -> y = [[-10, 40], [-1, 12]]; gamma_y = 40; scale = 3.175
    assert y.tolist() == [[-10.0, 40.0], [-1.0, 12.0]]
    assert gy.tolist() == [40.0] and sy[0] == np.float32(127.0) / np.float32(40.0)
    # -10 * 3.175 = -31.75 -> -32; 40 -> 127; -1 -> -3.175 -> -3; 12 -> 38.1 -> 38
    assert q.tolist() == [[-32, 127], [-3, 38]]


def test_dequantised_output_is_the_real_convolution(oracle):
    """y equals sum_k (x * gamma_x / 127) * (w * alpha) as real numbers, to three binary32
    roundings (the quotient and the two products)."""
    x, w, alpha, gamma_x = _case(1, 3, 10, 24, 16)
    q, gy, sy, y = oracle.conv_dyn(x, w, alpha, gamma_x, 10)
    xr = x.astype(np.float64).reshape(3, 10, 24) * (gamma_x.astype(np.float64) / 127.0)[:, None, None]
    wr = w.astype(np.float64) * alpha.astype(np.float64)[:, None]
    want = np.einsum("brk,ok->bro", xr, wr).reshape(30, 16)
    assert np.allclose(y, want, rtol=3 * 2.0 ** -23, atol=0)
    # and the maximum and the codes follow from y by the activation quantiser's definition
    q2, g2, s2 = oracle.quantize_act_absmax(y.reshape(3, -1))
    assert np.array_equal(q2.reshape(30, 16), q) and np.array_equal(g2, gy) and np.array_equal(s2, sy)


def test_identity_scales_in_exact_rationals(oracle):
    """alpha = 1 and gamma_x = 127 make y the integer accumulator itself; away from ties the
    codes are round(acc * 127 / max|acc|) as rational numbers."""
    x, w, _, _ = _case(2, 2, 6, 16, 8)
    q, gy, _, y = oracle.conv_dyn(x, w, np.ones(8, np.float32), np.full(2, 127.0, np.float32), 6)
    acc = x.astype(np.int64) @ w.astype(np.int64).T
    assert np.array_equal(y, acc.astype(np.float32))
    for b in range(2):
        blk = acc[b * 6:(b + 1) * 6]
        g = int(np.abs(blk).max())
        assert gy[b] == g
        for r in range(6):
            for o in range(8):
                v = Fraction(int(blk[r, o]) * 127, g)
                frac = v - (v.numerator // v.denominator)
                if abs(frac - Fraction(1, 2)) < Fraction(1, 500):
                    continue
                want = (v + Fraction(1, 2)).numerator // (v + Fraction(1, 2)).denominator
                assert int(q[b * 6 + r, o]) == want


def test_what_scales_change(oracle):
    x, w, alpha, gamma_x = _case(3, 2, 8, 32, 24)
    q, gy, sy, y = oracle.conv_dyn(x, w, alpha, gamma_x, 8)
    # a power of two on every alpha: same codes, gamma_y scaled (exact in binary32)
    q2, gy2, _, _ = oracle.conv_dyn(x, w, alpha * np.float32(4.0), gamma_x, 8)
    assert np.array_equal(q2, q) and np.array_equal(gy2, gy * 4)
    # a power of two on a sample's input scale: that sample's codes stay, its gamma_y scales
    gx2 = gamma_x.copy(); gx2[1] *= np.float32(0.5)
    q3, gy3, _, _ = oracle.conv_dyn(x, w, alpha, gx2, 8)
    assert np.array_equal(q3, q) and gy3[0] == gy[0] and gy3[1] == gy[1] * np.float32(0.5)
    # negating the weights of a channel negates its column
    w2 = w.copy(); w2[5] = -w2[5]
    q4, gy4, _, _ = oracle.conv_dyn(x, w2, alpha, gamma_x, 8)
    assert np.array_equal(q4[:, 5].astype(np.int32), -q[:, 5].astype(np.int32)) and np.array_equal(gy4, gy)
    assert np.array_equal(np.delete(q4, 5, axis=1), np.delete(q, 5, axis=1))
    # raising one channel's alpha above the rest moves the maximum there
    a5 = alpha.copy(); a5[7] = np.float32(50.0)
    q5, gy5, _, y5 = oracle.conv_dyn(x, w, a5, gamma_x, 8)
    for b in range(2):
        assert gy5[b] == np.abs(y5[b * 8:(b + 1) * 8, 7]).max()


def test_samples_are_independent_and_zero_input(oracle):
    x, w, alpha, gamma_x = _case(4, 3, 5, 16, 8)
    q, gy, sy, _ = oracle.conv_dyn(x, w, alpha, gamma_x, 5)
    for b in range(3):
        qb, gb, sb, _ = oracle.conv_dyn(x[b * 5:(b + 1) * 5], w, alpha, gamma_x[b:b + 1], 5)
        assert np.array_equal(qb, q[b * 5:(b + 1) * 5]) and gb[0] == gy[b] and sb[0] == sy[b]
    z = np.zeros((5, 16), np.int8)
    qz, gz, sz, _ = oracle.conv_dyn(z, w, alpha, np.array([0.0], np.float32), 5)
    assert not qz.any() and gz[0] == 0.0 and sz[0] == np.float32(127.0) / np.float32(1e-5)
