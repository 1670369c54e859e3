"""The allocation-free add/sub entry point against the ordinary one and the oracle.

Some callers of this library cannot let it allocate device memory: a serving
process whose memory pool already owns every free byte, or a plug-in that
runs inside another engine's arena, would see cudaMalloc fail or stall the
whole device.  `prom_pw_conv_i8_addsub_static` keeps the add/sub variant's
index lists in an array built into the library instead.  Here it is called
through the C ABI several times in a row, on different layers so that each
call finds the previous one's lists still in the shared array, and each result
must equal, byte for byte, both what `prom_pw_conv_i8` gives with the ADDSUB
variant and what the CPU oracle computes.  This file is collected last on
purpose: a run that stops at the first failure has then already been through
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth
from gpu_util import Guarded

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    yield
    assert binding.last_device_status() == binding.PROM_OK


def _layer(seed, m, cin, cout, zero_frac):
    x = synth.act_uniform_i8(seed, (m, cin), device="cuda")
    lay = synth.make_layer(seed, cin, cout, zero_frac, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
    return x, wp, rq, lay


def _oracle(oracle, x, lay):
    return oracle.conv_mul(x.cpu().numpy(), lay["w"].cpu().numpy(), lay["bias"].cpu().numpy(),
                           lay["mult"].cpu().numpy(), lay["shift"].cpu().numpy())


def test_calls_in_a_row_match_the_allocating_variant_and_the_oracle(oracle):
    # a wide layer first, then a narrower one with fewer non-zero weights (its lists are
    # shorter than what the first call left behind in the array), then a layer whose lists
    # take 2.4 MiB and whose staged rows need the large shared-memory launch, then a channel
    # count that is not a multiple of four (bytes are stored one by one)
    cases = [(61, 1000, 384, 96, 0.3), (62, 517, 144, 40, 0.7), (63, 260, 960, 320, 0.5),
             (64, 333, 64, 37, 0.5)]
    for seed, m, cin, cout, z in cases:
        x, wp, rq, lay = _layer(seed, m, cin, cout, z)
        want = torch.full((m, cout), -77, dtype=torch.int8, device="cuda")
        binding.pw_conv_i8(x, wp, cout, rq, y=want, variant="addsub")
        g = Guarded(m * cout, fill=55)
        got = g.view(m, cout)
        binding.pw_conv_i8_addsub_static(x, wp, cout, rq, y=got)
        g.check("output of the allocation-free entry point")
        assert torch.equal(got, want), (m, cin, cout)
        assert np.array_equal(got.cpu().numpy(), _oracle(oracle, x, lay)), (m, cin, cout)
    # and the first layer once more, now on top of the last one's lists
    seed, m, cin, cout, z = cases[0]
    x, wp, rq, lay = _layer(seed, m, cin, cout, z)
    want = binding.pw_conv_i8(x, wp, cout, rq, variant="addsub")
    got = binding.pw_conv_i8_addsub_static(x, wp, cout, rq)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    assert np.array_equal(got.cpu().numpy(), _oracle(oracle, x, lay))


def test_empty_input_is_a_no_op_with_any_pointers():
    x, wp, rq, _ = _layer(65, 4, 32, 48, 0.5)
    y = torch.full((0, 48), 7, dtype=torch.int8, device="cuda")
    binding.pw_conv_i8_addsub_static(x[:0], wp, 48, rq, y=y)
    rc = binding.lib().prom_pw_conv_i8_addsub_static(None, 0, 32, wp.data_ptr(), 48, rq, None, None)
    assert rc == binding.PROM_OK


def test_layer_beyond_the_built_in_scratch_is_refused():
    cin, cout = 1536, 1280          # needs about 7.5 MiB of lists: more than the array holds
    need = (cout * 16 + 255) // 256 * 256 + 4 * cout * (8 * ((cin + 7) // 8) + 8)
    assert need > binding.STATIC_SCRATCH_BYTES
    x = torch.zeros((8, cin), dtype=torch.int8, device="cuda")
    wp = torch.zeros((cout, cin // 4), dtype=torch.uint8, device="cuda")
    rq = binding.make_requant(torch.zeros(cout, dtype=torch.int32, device="cuda"),
                              torch.full((cout,), 1 << 30, dtype=torch.int32, device="cuda"),
                              torch.zeros(cout, dtype=torch.int8, device="cuda"))
    with pytest.raises(binding.PromError) as e:
        binding.pw_conv_i8_addsub_static(x, wp, cout, rq)
    assert e.value.code == binding.PROM_ERR_WORKSPACE
