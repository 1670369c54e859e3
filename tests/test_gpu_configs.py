"""GPU parity on the benchmark's single-layer configurations at their full sizes.

The compute-heavier late layers (three shapes at M = 25 088) against the whole-tensor
oracle, and the shape and sparsity sweep: every (Cin, Cout) pair at M = 12 544 with all four
zero fractions, the tensor-core variant (or what AUTO runs where it refuses the shape) and
the add/sub variant, whole tensor against the oracle; at M = 200 704 and 1 605 632 the corner
pairs plus 960 -> 1280, checked by the oracle on sampled rows (rows are independent, so a
sampled row is checked exactly) and against the plain one-thread-per-output kernel on the
whole tensor.  Every output lies between two bands of canary bytes.
"""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth
from gpu_util import Guarded, first_mismatch, sample_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    yield
    assert binding.last_device_status() == binding.PROM_OK


def _run(x, wp, cout, rq, variant):
    """(output tensor, variant that ran): an explicit variant that refuses the shape is
    replaced by AUTO and labelled so."""
    g = Guarded(x.shape[0] * cout)
    y = g.view(x.shape[0], cout)
    ran = variant
    try:
        binding.pw_conv_i8(x, wp, cout, rq, y=y, variant=variant)
    except binding.PromError as e:
        assert e.code == binding.PROM_ERR_UNSUPPORTED, (variant, e)
        ran = "auto"
        binding.pw_conv_i8(x, wp, cout, rq, y=y, variant="auto")
    g.check(f"output of {ran}")
    return y, ran


def _oracle_rows(oracle, x_rows, lay):
    return oracle.conv_mul(x_rows, lay["w"].cpu().numpy(), lay["bias"].cpu().numpy(),
                           lay["mult"].cpu().numpy(), lay["shift"].cpu().numpy())


@pytest.mark.parametrize("cin,cout", synth.CONFIG4_SHAPES)
def test_late_layers_at_batch_512_whole_tensor(oracle, cin, cout):
    m = 512 * 7 * 7
    seed = synth.BASE_SEED + 4
    x = synth.act_uniform_0_127(seed, (m, cin), device="cuda")
    lay = synth.make_layer(seed, cin, cout, 0.5, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
    want = _oracle_rows(oracle, x.cpu().numpy(), lay)
    for variant in ("tc", "auto", "addsub"):
        y, ran = _run(x, wp, cout, rq, variant)
        assert ran == variant
        assert first_mismatch(y.cpu().numpy(), want) is None, (cin, cout, variant)


@pytest.mark.parametrize("cin", synth.CONFIG5_CIN)
@pytest.mark.parametrize("cout", synth.CONFIG5_COUT)
def test_sweep_grid_smallest_m_whole_tensor(oracle, cin, cout):
    """All four zero fractions, both timed variants, every output against the oracle."""
    m = synth.CONFIG5_M[0]
    seed = synth.BASE_SEED + 5
    x = synth.act_uniform_i8(seed, (m, cin), device="cuda")
    xh = x.cpu().numpy()
    for z in synth.CONFIG5_ZERO:
        lay = synth.make_layer(seed, cin, cout, z, device="cuda")
        wp = binding.pack_ternary(lay["w"])
        rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
        want = _oracle_rows(oracle, xh, lay)
        for variant in ("tc", "addsub"):
            y, ran = _run(x, wp, cout, rq, variant)
            assert first_mismatch(y.cpu().numpy(), want) is None, (cin, cout, z, variant, ran)


LARGE_PAIRS = [(16, 24), (16, 1280), (960, 24), (960, 1280), (144, 320)]


@pytest.mark.parametrize("m", synth.CONFIG5_M[1:])
@pytest.mark.parametrize("pair", range(len(LARGE_PAIRS)))
def test_sweep_corners_large_m(oracle, m, pair):
    """The corner pairs of the grid and one interior pair at the two large M: sampled rows
    against the oracle, the whole tensor against the plain kernel (itself checked against the
    oracle on the same sampled rows).  The zero fraction rotates over the four of the sweep."""
    cin, cout = LARGE_PAIRS[pair]
    z = synth.CONFIG5_ZERO[(pair + (m > 300000)) % 4]
    seed = synth.BASE_SEED + 5
    x = synth.act_uniform_i8(seed, (m, cin), device="cuda")
    lay = synth.make_layer(seed, cin, cout, z, device="cuda")
    wp = binding.pack_ternary(lay["w"])
    rq = binding.make_requant(lay["bias"], lay["mult"], lay["shift"])
    rows = sample_rows(m, seed=pair)
    rows_d = torch.from_numpy(rows).cuda()
    want = _oracle_rows(oracle, x[rows_d].cpu().numpy(), lay)
    y_tc, ran = _run(x, wp, cout, rq, "tc")
    assert first_mismatch(y_tc[rows_d].cpu().numpy(), want) is None, (m, cin, cout, z, ran)
    y_nv, _ = _run(x, wp, cout, rq, "naive")
    assert first_mismatch(y_nv[rows_d].cpu().numpy(), want) is None, (m, cin, cout, z, "naive")
    assert torch.equal(y_tc, y_nv), (m, cin, cout, z, ran)
    del y_nv
    y_as, _ = _run(x, wp, cout, rq, "addsub")
    assert torch.equal(y_as, y_tc), (m, cin, cout, z, "addsub")
