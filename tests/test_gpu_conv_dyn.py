"""GPU parity of prom_pw_conv_i8_dyn (the pointwise layer in the paper's inference dataflow:
integer convolution, dequantised, quantised again per sample) with the CPU oracle: codes,
gamma_y and scale_y bit for bit, over several tiles, ragged tails, samples that end inside a
warp's 32 rows, wide and narrow channel counts; and chained after the activation quantiser."""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding

pytestmark = pytest.mark.gpu


def _case(seed, batch, rows, cin, cout, zero_frac=0.4):
    rng = np.random.default_rng(seed)
    x = rng.integers(-127, 128, size=(batch * rows, cin)).astype(np.int8)
    x[rng.random(x.shape) < 0.3] = 0
    w = rng.integers(-1, 2, size=(cout, cin)).astype(np.int8)
    w[rng.random(w.shape) < zero_frac] = 0
    alpha = rng.uniform(0.01, 0.2, size=cout).astype(np.float32)
    gamma_x = (rng.uniform(0.5, 8.0, size=batch) * 2.0 ** rng.integers(-6, 6, size=batch)).astype(np.float32)
    return x, w, alpha, gamma_x


def _run(oracle, x, w, alpha, gamma_x, rows):
    batch = gamma_x.shape[0]
    want_q, want_g, want_s, _ = oracle.conv_dyn(x, w, alpha, gamma_x, rows)
    wp = binding.pack_ternary(torch.from_numpy(w).cuda())
    q, g, s = binding.pw_conv_i8_dyn(torch.from_numpy(x).cuda(), batch, wp, w.shape[0],
                                     torch.from_numpy(alpha).cuda(), torch.from_numpy(gamma_x).cuda())
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    assert np.array_equal(g.cpu().numpy().view(np.uint32), want_g.view(np.uint32))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    got = q.cpu().numpy()
    bad = np.argwhere(got != want_q)
    assert len(bad) == 0, (len(bad), bad[:5].tolist(), got[tuple(bad[0])], want_q[tuple(bad[0])])


@pytest.mark.parametrize("batch,rows,cin,cout", [
    (2, 64, 16, 96),          # one tile, two samples inside it
    (3, 196, 64, 384),        # 14x14 images: samples end inside a warp's rows, several subtiles
    (5, 49, 160, 960),        # 7x7 images, wide output, K in two chunks
    (2, 3136, 32, 192),       # 56x56: many tiles per sample
    (4, 784, 96, 24),         # narrow output (one 16 + one 8 column piece)
    (1, 300, 384, 64),        # ragged last tile, K in three chunks
    (7, 1, 64, 40),           # one row per sample
])
def test_matches_the_oracle(oracle, batch, rows, cin, cout):
    _run(oracle, *_case(21, batch, rows, cin, cout), rows)


def test_after_the_activation_quantiser(oracle):
    """Float activations -> prom_quantize_act_absmax -> prom_pw_conv_i8_dyn, against the two
    oracle functions chained the same way."""
    rng = np.random.default_rng(22)
    batch, hw, cin, cout = 3, 28, 32, 192
    xf = rng.standard_normal((batch, hw, hw, cin)).astype(np.float32) * np.float32(3.0)
    w = rng.integers(-1, 2, size=(cout, cin)).astype(np.int8)
    alpha = rng.uniform(0.02, 0.1, size=cout).astype(np.float32)
    xq, gx, _ = oracle.quantize_act_absmax(xf)
    want_q, want_g, want_s, _ = oracle.conv_dyn(xq.reshape(-1, cin), w, alpha, gx, hw * hw)
    dq, dg, _ = binding.quantize_act_absmax(torch.from_numpy(xf).cuda())
    wp = binding.pack_ternary(torch.from_numpy(w).cuda())
    q, g, s = binding.pw_conv_i8_dyn(dq.reshape(-1, cin), batch, wp, cout, torch.from_numpy(alpha).cuda(), dg)
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), want_q)
    assert np.array_equal(g.cpu().numpy(), want_g) and np.array_equal(s.cpu().numpy(), want_s)


def test_refusals_and_degenerate_inputs(oracle):
    x, w, alpha, gx = _case(23, 2, 32, 24, 48)             # cin not a multiple of 16
    wp = binding.pack_ternary(torch.from_numpy(w).cuda())
    with pytest.raises(binding.PromError) as e:
        binding.pw_conv_i8_dyn(torch.from_numpy(x).cuda(), 2, wp, 48, torch.from_numpy(alpha).cuda(),
                               torch.from_numpy(gx).cuda())
    assert e.value.code == binding.PROM_ERR_UNSUPPORTED
    # an all-zero input: gamma_y = 0, scale = 127 / eps, every code 0
    x, w, alpha, gx = _case(24, 2, 100, 32, 64)
    x[:100] = 0
    _run(oracle, x, w, alpha, gx, 100)
    # twice in a row on the same buffers
    _run(oracle, x, w, alpha, gx, 100)


def test_seeded_shape_fuzz(oracle):
    rng = np.random.default_rng(98)
    for case in range(16):
        batch = int(rng.integers(1, 9)); rows = int(rng.integers(1, 700))
        cin = 16 * int(rng.integers(1, 25)); cout = 8 * int(rng.integers(1, 33))
        _run(oracle, *_case(200 + case, batch, rows, cin, cout), rows)
