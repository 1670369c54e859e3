"""Pins of the oracle's int8 depthwise 3x3 convolution: closed forms on constant images
(interior, edge and corner sums under zero padding), the identity and shift kernels, an
independent formulation with an explicitly padded array and array slices, the relation between
stride 2 and stride 1, linearity in the weights, and the requantiser shared with the pointwise
layers."""
import numpy as np
import pytest


def _unit(c):
    # requantisation that halves: with a centre weight of 2 the layer is the identity
    return np.zeros(c, np.int32), np.full(c, 1 << 30, np.int32), np.zeros(c, np.int8)


def test_constant_image_closed_form(oracle):
    c = 4
    x = np.full((1, 5, 6, c), 3, np.int8)
    w = np.ones((c, 3, 3), np.int8)
    _, acc = oracle.dw3x3(x, w, *_unit(c), want_acc=True)
    assert acc.shape == (1, 5, 6, c)
    assert (acc[0, 1:-1, 1:-1] == 27).all()                       # 9 taps inside
    assert (acc[0, 0, 1:-1] == 18).all() and (acc[0, 1:-1, 0] == 18).all()   # 6 taps on an edge
    assert (acc[0, 0, 0] == 12).all() and (acc[0, -1, -1] == 12).all()       # 4 taps in a corner


def test_identity_and_shift_kernels(oracle):
    rng = np.random.default_rng(1)
    c = 8
    x = rng.integers(-128, 128, size=(2, 7, 9, c)).astype(np.int8)
    w = np.zeros((c, 3, 3), np.int8); w[:, 1, 1] = 2
    assert np.array_equal(oracle.dw3x3(x, w, *_unit(c)), x)
    # tap (0, 1) reads the pixel above: the image moves down by one row, zeros enter at the top
    w = np.zeros((c, 3, 3), np.int8); w[:, 0, 1] = 2
    y = oracle.dw3x3(x, w, *_unit(c))
    assert np.array_equal(y[:, 1:], x[:, :-1]) and not y[:, 0].any()
    # tap (1, 2) reads the pixel to the right: the image moves left
    w = np.zeros((c, 3, 3), np.int8); w[:, 1, 2] = 2
    y = oracle.dw3x3(x, w, *_unit(c))
    assert np.array_equal(y[:, :, :-1], x[:, :, 1:]) and not y[:, :, -1].any()


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("h,w", [(6, 6), (7, 5), (1, 4)])
def test_against_padded_slices(oracle, stride, h, w):
    """The same sums written with an explicitly padded int64 array and nine strided slices."""
    rng = np.random.default_rng(2)
    c = 5
    x = rng.integers(-128, 128, size=(2, h, w, c)).astype(np.int8)
    wt = rng.integers(-128, 128, size=(c, 3, 3)).astype(np.int8)
    _, acc = oracle.dw3x3(x, wt, *_unit(c), stride=stride, want_acc=True)
    xp = np.zeros((2, h + 2, w + 2, c), np.int64); xp[:, 1:-1, 1:-1] = x
    ho, wo = (h - 1) // stride + 1, (w - 1) // stride + 1
    want = np.zeros((2, ho, wo, c), np.int64)
    for di in range(3):
        for dj in range(3):
            want += xp[:, di:di + (ho - 1) * stride + 1:stride, dj:dj + (wo - 1) * stride + 1:stride] * \
                    wt[:, di, dj].astype(np.int64)
    assert np.array_equal(acc, want)


def test_stride_two_is_stride_one_subsampled(oracle):
    rng = np.random.default_rng(3)
    c = 6
    x = rng.integers(-128, 128, size=(1, 9, 8, c)).astype(np.int8)
    wt = rng.integers(-20, 20, size=(c, 3, 3)).astype(np.int8)
    rq = (rng.integers(-100, 100, size=c).astype(np.int32), np.full(c, 1 << 30, np.int32), np.full(c, 4, np.int8))
    y1 = oracle.dw3x3(x, wt, *rq, stride=1)
    y2 = oracle.dw3x3(x, wt, *rq, stride=2)
    assert np.array_equal(y2, y1[:, ::2, ::2])


def test_linear_in_the_weights_and_channels_do_not_mix(oracle):
    rng = np.random.default_rng(4)
    c = 4
    x = rng.integers(-128, 128, size=(1, 6, 6, c)).astype(np.int8)
    wa = rng.integers(-60, 60, size=(c, 3, 3)).astype(np.int8)
    wb = rng.integers(-60, 60, size=(c, 3, 3)).astype(np.int8)
    _, a = oracle.dw3x3(x, wa, *_unit(c), want_acc=True)
    _, b = oracle.dw3x3(x, wb, *_unit(c), want_acc=True)
    _, ab = oracle.dw3x3(x, (wa + wb).astype(np.int8), *_unit(c), want_acc=True)
    assert np.array_equal(ab, a + b)
    # changing channel 2's input or filter leaves the other channels alone
    x2 = x.copy(); x2[..., 2] = 0
    _, a2 = oracle.dw3x3(x2, wa, *_unit(c), want_acc=True)
    assert np.array_equal(np.delete(a2, 2, axis=3), np.delete(a, 2, axis=3)) and not a2[..., 2].any()


def test_requantiser_is_the_pointwise_one(oracle):
    rng = np.random.default_rng(5)
    c = 3
    x = rng.integers(-128, 128, size=(1, 4, 4, c)).astype(np.int8)
    wt = rng.integers(-128, 128, size=(c, 3, 3)).astype(np.int8)
    bias = np.array([5, -7, 1000], np.int32); mult = np.array([1 << 30, 1500000000, 2000000000], np.int32)
    shift = np.array([3, 6, 9], np.int8)
    y, acc = oracle.dw3x3(x, wt, bias, mult, shift, act_min=0, act_max=127, want_acc=True)
    for ch in range(c):
        want = oracle.requant((acc[..., ch] + bias[ch]).ravel(), int(mult[ch]), int(shift[ch]), 0, 127)
        assert np.array_equal(y[..., ch].ravel(), want.astype(np.int8))
