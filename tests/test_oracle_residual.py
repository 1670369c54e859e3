"""Pins of the oracle's skip connection (Section 2): every pair of int8 values against Python
integers, the cases that saturate, zero as the identity, symmetry in the operands, and the
difference from an addition that wraps around."""
import numpy as np


def test_every_pair_of_int8_values(oracle):
    a, b = np.meshgrid(np.arange(-128, 128), np.arange(-128, 128), indexing="ij")
    got = oracle.residual_add(a.astype(np.int8), b.astype(np.int8))
    want = [[max(-128, min(127, i + j)) for j in range(-128, 128)] for i in range(-128, 128)]
    assert got.dtype == np.int8 and got.tolist() == want


def test_saturation_and_identity(oracle):
    a = np.array([127, 127, -128, -128, 100, -100, 5, 0], np.int8)
    b = np.array([1, 127, -1, -128, 27, -28, -5, 0], np.int8)
    assert oracle.residual_add(a, b).tolist() == [127, 127, -128, -128, 127, -128, 0, 0]
    x = np.arange(-128, 128).astype(np.int8)
    assert np.array_equal(oracle.residual_add(x, np.zeros_like(x)), x)
    assert np.array_equal(oracle.residual_add(np.zeros_like(x), x), x)


def test_symmetric_and_not_wrapping(oracle):
    rng = np.random.default_rng(7)
    a = rng.integers(-128, 128, size=(3, 5, 7, 8)).astype(np.int8)
    b = rng.integers(-128, 128, size=(3, 5, 7, 8)).astype(np.int8)
    s = oracle.residual_add(a, b)
    assert s.shape == a.shape and np.array_equal(s, oracle.residual_add(b, a))
    total = a.astype(np.int16) + b
    wrapped = total.astype(np.int8)                                 # two's-complement wrap-around
    over = (total > 127) | (total < -128)
    assert over.any() and (s[over] != wrapped[over]).all()
    assert np.array_equal(s[~over], wrapped[~over])
