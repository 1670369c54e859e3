"""Pins for the oracle's accumulation: brute force, identities, special cases,
a library matmul.  Each would fail on a dropped term, a wrong sign, a
transposed operand or a wrong index."""
import itertools

import numpy as np
import torch

IDENT = dict(act_min=-128, act_max=127)


def ident_requant(cout):
    """bias 0, mult 2^30, shift 0  ->  q = rha(acc / 2)."""
    return (np.zeros(cout, np.int32), np.full(cout, 1 << 30, np.int32), np.zeros(cout, np.int8))


def py_acc(x, w):
    """Python big-int evaluation of sum_k x[m][k]*w[o][k]."""
    return [[sum(int(a) * int(b) for a, b in zip(xr, wo)) for wo in w] for xr in x]


def test_brute_force_all_ternary_matrices(oracle):
    rng = np.random.default_rng(0)
    for cout, cin in [(1, 1), (2, 2), (1, 5), (3, 2), (2, 4), (4, 2)]:
        x = rng.integers(-128, 128, size=(5, cin), dtype=np.int8)
        x[0, :] = -128
        x[1, :] = 127
        b, m, s = ident_requant(cout)
        for flat in itertools.product((-1, 0, 1), repeat=cout * cin):
            w = np.array(flat, dtype=np.int8).reshape(cout, cin)
            _, acc = oracle.conv_mul(x, w, b, m, s, want_acc=True, **IDENT)
            assert acc.tolist() == py_acc(x.tolist(), w.tolist())
            _, acc2 = oracle.conv_addsub(x, w, b, m, s, want_acc=True, **IDENT)
            assert acc2.tolist() == acc.tolist()


def test_mul_form_equals_addsub_form(oracle):
    rng = np.random.default_rng(1)
    for m, cin, cout in [(7, 16, 24), (33, 24, 144), (5, 960, 8), (64, 145, 37)]:
        x = rng.integers(-128, 128, size=(m, cin), dtype=np.int8)
        w = rng.integers(-1, 2, size=(cout, cin), dtype=np.int8)
        bias = rng.integers(-4096, 4097, size=cout).astype(np.int32)
        mult = rng.integers(1 << 30, 1 << 31, size=cout).astype(np.int32)
        shift = rng.integers(0, 13, size=cout).astype(np.int8)
        y1, a1 = oracle.conv_mul(x, w, bias, mult, shift, -128, 127, want_acc=True)
        y2, a2 = oracle.conv_addsub(x, w, bias, mult, shift, -128, 127, want_acc=True)
        assert np.array_equal(a1, a2) and np.array_equal(y1, y2)


def test_against_int64_matmul_and_float64_conv2d(oracle):
    rng = np.random.default_rng(2)
    b, h, wd, cin, cout = 2, 5, 3, 48, 20
    x = rng.integers(-128, 128, size=(b, h, wd, cin), dtype=np.int8)
    w = rng.integers(-1, 2, size=(cout, cin), dtype=np.int8)
    bi, mu, sh = ident_requant(cout)
    _, acc = oracle.conv_mul(x.reshape(-1, cin), w, bi, mu, sh, want_acc=True, **IDENT)
    want = torch.from_numpy(x.reshape(-1, cin)).to(torch.int64) @ torch.from_numpy(w).to(torch.int64).T
    assert np.array_equal(acc, want.numpy())
    # the same layer as a 1x1 convolution over NCHW data (the paper's layout)
    xc = torch.from_numpy(x).permute(0, 3, 1, 2).to(torch.float64)
    wc = torch.from_numpy(w).to(torch.float64).view(cout, cin, 1, 1)
    yc = torch.nn.functional.conv2d(xc, wc).permute(0, 2, 3, 1).reshape(-1, cout)
    assert np.array_equal(acc.astype(np.float64), yc.numpy())


def test_zero_weights_give_bias_only(oracle):
    rng = np.random.default_rng(3)
    x = rng.integers(-128, 128, size=(9, 32), dtype=np.int8)
    w = np.zeros((6, 32), np.int8)
    bias = np.array([0, 256, 511, 512, -256, 40000], np.int32)
    mult = np.full(6, 1 << 30, np.int32)
    shift = np.full(6, 8, np.int8)          # scale 2^-9
    y, acc = oracle.conv_mul(x, w, bias, mult, shift, -128, 127, want_acc=True)
    assert not acc.any()
    # rha(bias/512): 0, 0.5->1, 0.998->1, 1, -0.5->-1, 78.1->78
    assert y.tolist() == [[0, 1, 1, 1, -1, 78]] * 9


def test_one_hot_weight_reproduces_the_channel(oracle):
    rng = np.random.default_rng(4)
    cin, cout = 40, 40
    x = rng.integers(-128, 128, size=(11, cin), dtype=np.int8)
    perm = rng.permutation(cin)
    w = np.zeros((cout, cin), np.int8)
    w[np.arange(cout), perm] = 1
    bi, mu, sh = ident_requant(cout)
    _, acc = oracle.conv_mul(x, w, bi, mu, sh, want_acc=True, **IDENT)
    assert np.array_equal(acc, x[:, perm].astype(np.int32))
    # two equal input channels, both weighted +1, scale 1/2  ->  y = x
    x2 = np.concatenate([x, x], axis=1)
    w2 = np.concatenate([w, w], axis=1)
    y = oracle.conv_mul(x2, w2, bi, mu, sh, **IDENT)
    assert np.array_equal(y, x[:, perm])
    # -1 on the one-hot position negates
    _, accn = oracle.conv_mul(x, -w, bi, mu, sh, want_acc=True, **IDENT)
    assert np.array_equal(accn, -acc)


def test_permuting_k_leaves_the_result_unchanged(oracle):
    rng = np.random.default_rng(5)
    m, cin, cout = 13, 64, 17
    x = rng.integers(-128, 128, size=(m, cin), dtype=np.int8)
    w = rng.integers(-1, 2, size=(cout, cin), dtype=np.int8)
    bias = rng.integers(-4096, 4097, size=cout).astype(np.int32)
    mult = rng.integers(1 << 30, 1 << 31, size=cout).astype(np.int32)
    shift = rng.integers(8, 13, size=cout).astype(np.int8)
    p = rng.permutation(cin)
    y1 = oracle.conv_mul(x, w, bias, mult, shift)
    y2 = oracle.conv_mul(x[:, p], w[:, p], bias, mult, shift)
    assert np.array_equal(y1, y2)
    # rows of X are independent; channels of W are independent
    y3 = oracle.conv_mul(x[::-1], w[::-1], bias[::-1], mult[::-1], shift[::-1])
    assert np.array_equal(y3, y1[::-1, ::-1])


def test_extreme_accumulator(oracle):
    # |acc| reaches 960*128 without wrapping anything
    x = np.full((2, 960), -128, np.int8)
    w = np.ones((2, 960), np.int8)
    w[1] = -1
    bi, mu, sh = ident_requant(2)
    _, acc = oracle.conv_mul(x, w, bi, mu, sh, want_acc=True, **IDENT)
    assert acc.tolist() == [[-122880, 122880]] * 2
