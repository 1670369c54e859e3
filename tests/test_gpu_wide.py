"""GPU parity of the row-resident tensor-core kernel (contraction-bound layers).

The kernel is forced through `prom_debug_tc_wide(2)` on shapes that cover: one and several K
chunks with a full and a partial last chunk, column tiles that end inside the first or the second
half of 128 channels, fewer row tiles than SMs (CTAs share a row tile's columns) and several row
tiles per CTA, a ragged last row tile, both epilogues (the one-multiply form and the 64-bit
definition, chosen per column tile) and both clamps.  Every output is compared with the CPU oracle
and lies between two bands of canary bytes.
"""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth
from gpu_util import first_mismatch, make_case, oracle_y, run_variant, sample_rows, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    binding.debug_tc_wide(2)
    yield
    binding.debug_tc_wide(0)
    assert binding.last_device_status() == binding.PROM_OK


SHAPES = [
    (1000, 128, 64),        # one chunk, half a column tile
    (333, 144, 96),         # second chunk of 16 bytes, a column tile that ends in its second half
    (2500, 384, 320),       # three column tiles, the last one half full
    (300, 960, 1280),       # K = 7.5 chunks, ten column tiles shared by the CTAs of a row tile
    (12544, 960, 1280),     # a point of the benchmark's sweep, whole tensor
    (37965, 256, 256),      # two and three row tiles per CTA, ragged end
    (5000, 1024, 128),      # the largest K
    (129, 208, 448),
    (40000, 512, 640),      # N = 256: two and a half column tiles, the resident rows at their limit
]


@pytest.fixture(params=[1, 2], ids=["n128", "n256"])
def blocks(request):
    """128-channel blocks per column tile: MMAs of N = 128 or N = 256."""
    binding.debug_tc_wide(2, request.param)
    yield request.param
    binding.debug_tc_wide(2, 0)


@pytest.mark.parametrize("m,cin,cout", SHAPES)
def test_matches_oracle(oracle, blocks, m, cin, cout):
    x, lay = make_case(7000 + cin + cout, m, cin, cout, 0.5, act="i8")
    xd, wp, consts = to_device(x, lay)
    if blocks == 2 and cin > 512:
        # four 32 KB stages do not fit beside the resident rows
        with pytest.raises(binding.PromError) as e:
            binding.pw_conv_i8(xd, wp, cout, binding.make_requant(*consts), variant="tc")
        assert e.value.code == binding.PROM_ERR_UNSUPPORTED
        return
    got = run_variant(xd, wp, consts, cout, "tc")
    assert binding.last_device_status() == binding.PROM_OK
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None, (m, cin, cout)


def test_same_bytes_as_the_weight_resident_kernel():
    m, cin, cout = 20000, 384, 1280
    x, lay = make_case(7100, m, cin, cout, 0.7, act="relu6")
    xd, wp, consts = to_device(x, lay)
    a = run_variant(xd, wp, consts, cout, "tc")
    try:
        binding.debug_tc_wide(1)
        b = run_variant(xd, wp, consts, cout, "tc")
    finally:
        binding.debug_tc_wide(2)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("lo,hi", [(-128, 127), (-5, 90), (0, 127)])
def test_clamps_and_wide_shift_spans(oracle, blocks, lo, hi):
    """Shifts 1..20 inside one column tile and a signed clamp: the 64-bit epilogue; the third case
    mixes a tile on the one-multiply form with tiles on the 64-bit form."""
    m, cin, cout = 3000, 256, 384
    x, lay = make_case(7200 + hi, m, cin, cout, 0.5, act="i8", shift_lo=1, shift_hi=20)
    if (lo, hi) == (0, 127):
        lay["shift"][:128] = 7                                  # first column tile: one shift, fast form
    xd, wp, consts = to_device(x, lay)
    got = run_variant(xd, wp, consts, cout, "tc", lo, hi)
    assert first_mismatch(got, oracle_y(oracle, x, lay, lo, hi)) is None


def test_large_m_sampled_rows(oracle, blocks):
    m, cin, cout = 200704, 384, 320
    seed = synth.BASE_SEED + 5
    x = synth.act_uniform_i8(seed, (m, cin), device="cuda")
    lay = synth.make_layer(seed, cin, cout, 0.5, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
    y = binding.pw_conv_i8(x, wp, cout, rq, variant="tc")
    y_nv = binding.pw_conv_i8(x, wp, cout, rq, variant="naive")
    torch.cuda.synchronize()
    assert torch.equal(y, y_nv)
    rows = torch.from_numpy(sample_rows(m, seed=3)).cuda()
    want = oracle.conv_mul(x[rows].cpu().numpy(), lay["w"].cpu().numpy(), lay["bias"].cpu().numpy(),
                           lay["mult"].cpu().numpy(), lay["shift"].cpu().numpy())
    assert first_mismatch(y[rows].cpu().numpy(), want) is None


def test_bad_constants_are_reported():
    m, cin, cout = 500, 128, 256
    x, lay = make_case(7300, m, cin, cout, 0.5)
    lay["mult"][130] = -5
    xd, wp, consts = to_device(x, lay)
    rq = binding.make_requant(*consts)
    binding.pw_conv_i8(xd, wp, cout, rq, variant="tc")
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_ERR_BAD_REQUANT


def test_shapes_it_cannot_take_are_refused():
    for m, cin, cout in [(1000, 64, 256), (1000, 1040, 256), (1000, 256, 48), (1000, 136, 256)]:
        x, lay = make_case(7400, m, cin, cout, 0.5)
        xd, wp, consts = to_device(x, lay)
        rq = binding.make_requant(*consts)
        with pytest.raises(binding.PromError) as e:
            binding.pw_conv_i8(xd, wp, cout, rq, variant="tc")
        assert e.value.code == binding.PROM_ERR_UNSUPPORTED
