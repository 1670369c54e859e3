"""GPU parity of prom_dw_conv3x3_i8 with the CPU oracle, byte for byte: both strides, odd and
even image sizes (padding on every side), strips that end inside the row, channel counts of
the network's hidden layers, both clamps, extreme values."""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding

pytestmark = pytest.mark.gpu


def _case(seed, b, h, w, c, extreme=False):
    rng = np.random.default_rng(seed)
    x = rng.integers(-128, 128, size=(b, h, w, c)).astype(np.int8)
    wt = rng.integers(-128, 128, size=(c, 3, 3)).astype(np.int8)
    if extreme:
        x[:] = -128; wt[:] = -128
    bias = rng.integers(-4096, 4097, size=c).astype(np.int32)
    mult = rng.integers(1 << 30, (1 << 31) - 1, size=c).astype(np.int32)
    shift = rng.integers(6, 12, size=c).astype(np.int8)
    return x, wt, bias, mult, shift


def _run(oracle, x, wt, bias, mult, shift, stride, lo, hi):
    want = oracle.dw3x3(x, wt, bias, mult, shift, stride=stride, act_min=lo, act_max=hi)
    rq = binding.make_requant(torch.from_numpy(bias).cuda(), torch.from_numpy(mult).cuda(),
                              torch.from_numpy(shift).cuda(), act_min=lo, act_max=hi)
    y = binding.dw_conv3x3_i8(torch.from_numpy(x).cuda(), torch.from_numpy(wt).cuda(), rq, stride=stride)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    got = y.cpu().numpy()
    assert got.shape == want.shape
    bad = np.argwhere(got != want)
    assert len(bad) == 0, (len(bad), bad[:5].tolist())


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("b,h,w,c", [
    (2, 14, 14, 96), (1, 7, 7, 960), (3, 28, 28, 144), (2, 9, 13, 32), (1, 1, 1, 16), (2, 5, 6, 4),
    (1, 56, 56, 24),
])
def test_matches_the_oracle(oracle, stride, b, h, w, c):
    _run(oracle, *_case(31, b, h, w, c), stride, 0, 127)


def test_signed_clamp_and_extreme_values(oracle):
    _run(oracle, *_case(32, 2, 10, 10, 64), 1, -128, 127)
    _run(oracle, *_case(33, 1, 6, 6, 32, extreme=True), 2, -128, 127)
    _run(oracle, *_case(33, 1, 6, 6, 32, extreme=True), 1, 0, 127)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("lo", [0, -128])
def test_small_and_mixed_shifts_and_large_biases(oracle, stride, lo):
    """Shifts 0..3 (below 2 the requantiser keeps two more bits of the product), mixed within a
    thread's four channels, small weights so that outputs stay inside the clamp, and biases up to
    the limit of 2^28 with shifts that bring them back into range."""
    rng = np.random.default_rng(36)
    b, h, w, c = 2, 11, 9, 48
    x = rng.integers(-128, 128, size=(b, h, w, c)).astype(np.int8)
    wt = rng.integers(-2, 3, size=(c, 3, 3)).astype(np.int8)
    bias = rng.integers(-300, 301, size=c).astype(np.int32)
    mult = rng.integers(1 << 28, (1 << 31) - 1, size=c).astype(np.int32)
    shift = (np.arange(c) % 4).astype(np.int8)
    _run(oracle, x, wt, bias, mult, shift, stride, lo, 127)
    shift[:] = rng.integers(0, 2, size=c)
    _run(oracle, x, wt, bias, mult, shift, stride, lo, 127)
    bias = (rng.integers(-(1 << 28), (1 << 28) + 1, size=c)).astype(np.int32)
    shift[:] = rng.integers(20, 24, size=c)
    _run(oracle, x, wt, bias, mult, shift, stride, lo, 127)


def test_refusals():
    x = torch.zeros((1, 4, 4, 6), dtype=torch.int8, device="cuda")
    w = torch.zeros((6, 3, 3), dtype=torch.int8, device="cuda")
    z = torch.zeros((6,), dtype=torch.int32, device="cuda")
    rq = binding.make_requant(z, z + (1 << 30), torch.zeros((6,), dtype=torch.int8, device="cuda"))
    with pytest.raises(binding.PromError) as e:
        binding.dw_conv3x3_i8(x, w, rq)
    assert e.value.code == binding.PROM_ERR_UNSUPPORTED


def test_seeded_shape_fuzz(oracle):
    rng = np.random.default_rng(99)
    for case in range(24):
        b = int(rng.integers(1, 4)); h = int(rng.integers(1, 40)); w = int(rng.integers(1, 40))
        c = 4 * int(rng.integers(1, 80))
        stride = int(rng.choice([1, 2]))
        lo, hi = (0, 127) if case % 2 else (-128, 127)
        _run(oracle, *_case(100 + case, b, h, w, c), stride, lo, hi)


@pytest.mark.parametrize("b,h,w,c", [
    (2, 14, 14, 96), (1, 7, 7, 960), (3, 28, 28, 144), (2, 9, 13, 32), (1, 16, 8, 16), (2, 33, 17, 64),
    (1, 56, 56, 48), (4, 5, 40, 80), (1, 1, 130, 16),
])
def test_stride_1_on_the_tensor_cores(oracle, b, h, w, c):
    """The TMA + tcgen05 form (stride 1, whole slices of 16 channels) forced, against the oracle
    and against the CUDA-core kernel: tiles that end inside the image on both axes, one to four
    slices per CTA, several channel groups, images smaller than a tile."""
    x, wt, bias, mult, shift = _case(41, b, h, w, c)
    try:
        for lo, hi in ((0, 127), (-128, 127), (3, 100)):
            binding.debug_dw_variant(2)
            _run(oracle, x, wt, bias, mult, shift, 1, lo, hi)
            binding.debug_dw_variant(1)
            _run(oracle, x, wt, bias, mult, shift, 1, lo, hi)
    finally:
        binding.debug_dw_variant(0)


def test_tensor_core_form_refuses_what_it_cannot_take():
    x = torch.zeros((1, 8, 8, 24), dtype=torch.int8, device="cuda")
    w = torch.zeros((24, 3, 3), dtype=torch.int8, device="cuda")
    z = torch.zeros((24,), dtype=torch.int32, device="cuda")
    rq = binding.make_requant(z, z + (1 << 30), torch.zeros((24,), dtype=torch.int8, device="cuda"))
    try:
        binding.debug_dw_variant(2)
        for stride in (1, 2):                       # 24 channels: no whole slices; stride 2: not built
            with pytest.raises(binding.PromError) as e:
                binding.dw_conv3x3_i8(x, w, rq, stride=stride)
            assert e.value.code == binding.PROM_ERR_UNSUPPORTED
    finally:
        binding.debug_dw_variant(0)
    binding.dw_conv3x3_i8(x, w, rq, stride=1)       # the library's choice still runs it
    torch.cuda.synchronize()
