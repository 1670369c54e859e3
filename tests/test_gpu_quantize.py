"""GPU parity of the ternary absmean quantiser (paper Eq. 1-3, Figure 10) against the
oracle, through the C ABI, and the quantise -> convolve chain."""
import math

import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    yield
    assert binding.last_device_status() == binding.PROM_OK


def check(oracle, w):
    """Codes must equal the oracle's except where the ratio W/alpha sits within 1e-9 of a
    rounding tie (the two sides add |W| in different orders, both in binary64); in practice
    there is no such element and the comparison is exact."""
    cout, cin = w.shape
    q, alpha = oracle.quantize_ternary(w.numpy())
    packed, a = binding.quantize_ternary(w.cuda())
    torch.cuda.synchronize()
    got, bad = oracle.unpack(packed.cpu().numpy(), cout, cin)
    assert bad == 0
    ratio = w.numpy().astype(np.float64) / np.maximum(alpha, 1e-5)[:, None]
    near_tie = np.minimum(np.abs(np.abs(ratio) - 0.5), np.abs(np.abs(ratio) - 1.5)) < 1e-9
    assert np.array_equal(got[~near_tie], q[~near_tie])
    assert np.allclose(a.cpu().numpy(), alpha.astype(np.float32), rtol=1e-6, atol=1e-12)
    return q, packed


@pytest.mark.parametrize("cout,cin", [(1, 1), (5, 3), (16, 24), (37, 145), (384, 64), (1280, 320), (96, 4096)])
def test_quantiser_matches_oracle(oracle, cout, cin):
    g = torch.Generator().manual_seed(cout * 7919 + cin)
    w = torch.randn((cout, cin), generator=g) * math.sqrt(2.0 / cout)     # He-normal, as the paper initialises
    check(oracle, w)


def test_quantiser_special_rows(oracle):
    w = torch.zeros((6, 8))
    w[0] = torch.tensor([0.5, -0.5, 1.5, -1.5, 2.5, 0.0, 0.25, 1.25])      # mean 1: exact ties
    w[1] = 3.0                                                              # ratio exactly 1
    w[2, 0], w[2, 1], w[2, 2] = 6e-6, 5.2e-6, 8e-6 - 11.2e-6 + 8e-6        # mean below eps
    w[3] = torch.tensor([1e30, -1e30, 1e-30, 0, 0, 0, 0, 0])
    w[5] = -w[0]
    q, _ = check(oracle, w)
    assert q[0].tolist() == [0, 0, 1, -1, 1, 0, 0, 1] and q[5].tolist() == [0, 0, -1, 1, -1, 0, 0, -1]


def test_quantise_then_convolve(oracle):
    """Float weights -> prom_quantize_ternary -> prom_pw_conv_i8 equals the oracle's
    quantiser followed by the oracle's convolution."""
    m, cin, cout = 700, 96, 160
    g = torch.Generator().manual_seed(9)
    w = torch.randn((cout, cin), generator=g) * math.sqrt(2.0 / cout)
    q, _ = oracle.quantize_ternary(w.numpy())
    x = synth.act_post_relu6(9, (m, cin))
    bias, mult, shift = synth.requant_constants(9, cout)
    want = oracle.conv_mul(x.numpy(), q, bias.numpy(), mult.numpy(), shift.numpy())
    packed, _ = binding.quantize_ternary(w.cuda())
    consts = (bias.cuda(), mult.cuda(), shift.cuda())
    y = binding.pw_conv_i8(x.cuda(), packed, cout, binding.make_requant(*consts))
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), want)


def test_nan_weight_is_reported():
    w = torch.ones((4, 8))
    w[1, 3] = float("nan")
    binding.quantize_ternary(w.cuda())
    assert binding.last_device_status() == binding.PROM_ERR_BAD_WEIGHT


def test_all_matrices_in_one_launch(oracle):
    """prom_quantize_ternary_batch over matrices of different shapes equals the per-matrix call
    and the oracle, codes and scales."""
    shapes = [(16, 32), (96, 16), (37, 145), (1, 1), (1280, 320), (24, 96), (5, 3)]
    g = torch.Generator().manual_seed(77)
    ws = [(torch.randn(s, generator=g) * math.sqrt(2.0 / s[0])).cuda() for s in shapes]
    outs = binding.quantize_ternary_batch(ws)
    torch.cuda.synchronize()
    for w, (packed, alpha) in zip(ws, outs):
        p1, a1 = binding.quantize_ternary(w)
        torch.cuda.synchronize()
        assert torch.equal(packed, p1) and torch.equal(alpha, a1)
        q, al = oracle.quantize_ternary(w.cpu().numpy())
        got, bad = oracle.unpack(packed.cpu().numpy(), *w.shape)
        assert bad == 0 and np.array_equal(got, q)
    # argument checks happen before anything is launched
    jobs = (binding.PromQuantizeJob * 1)(binding.PromQuantizeJob(ws[0].data_ptr(), 16, 32, outs[0][0].data_ptr(), 3, None))
    assert binding.lib().prom_quantize_ternary_batch(jobs, 1, None) == binding.PROM_ERR_WORKSPACE
    assert binding.lib().prom_quantize_ternary_batch(None, 1, None) == binding.PROM_ERR_NULL
