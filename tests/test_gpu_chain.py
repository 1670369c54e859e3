"""GPU parity of the depth-first launches inside a layer sequence.

A run of consecutive layers that `prom_pw_layer_seq` executes in one launch (a CTA takes
its tiles of rows through all the layers of the run) must still write every layer's output
to the workspace: each intermediate tensor is compared with the CPU oracle here, not only
the last one, and the result must not depend on whether the depth-first launches are used.
"""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth
from gpu_util import Guarded, first_mismatch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    binding.debug_seq_chain(1)
    yield
    binding.debug_seq_chain(0)
    assert binding.last_device_status() == binding.PROM_OK


def make_stack(seed, shapes, shift_span=None):
    """shapes: [(cin, cout, in_stride)]; returns (host layers for the oracle, LayerSeq)."""
    host, dev = [], []
    for i, (cin, cout, stride) in enumerate(shapes):
        d = synth.make_layer(seed, cin, cout, 0.5, index=i + 1)
        if shift_span is not None and i == shift_span:
            d["shift"][: max(1, cout // 3)] = 1          # a span above 4: the 64-bit epilogue
        host.append(dict(cin=cin, cout=cout, in_stride=stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                         mult=d["mult"].numpy(), shift=d["shift"].numpy()))
        dev.append(dict(cin=cin, cout=cout, in_stride=stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                        bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda()))
    return host, binding.LayerSeq(dev), dev


def oracle_intermediates(oracle, host, x0):
    """Every layer's output, by the oracle's single-layer functions applied in turn."""
    outs = []
    cur = x0
    for hl in host:
        if hl["in_stride"] != 1:
            cur = oracle.subsample(cur, hl["in_stride"])
        b, h, w, c = cur.shape
        cur = oracle.conv_mul(cur.reshape(-1, c), hl["w"], hl["bias"], hl["mult"], hl["shift"]).reshape(
            b, h, w, hl["cout"])
        outs.append(cur)
    return outs


def run_and_check_all(oracle, host, seq, x0, expect_chained=None):
    """Runs the sequence in a guarded workspace and compares the final output and every
    intermediate that a depth-first launch wrote with the oracle.  Returns the chained flags."""
    batch, h0, w0, _ = x0.shape
    want = oracle_intermediates(oracle, host, x0.numpy())
    nbytes = max(16, seq.workspace_bytes(batch, h0, w0))
    g = Guarded(nbytes, dtype=torch.uint8, fill=0xEE)
    ws = g.view(nbytes)
    gy = Guarded(want[-1].size)
    y = gy.view(*want[-1].shape)
    binding.pw_layer_seq(seq, x0.cuda(), ws, y_out=y)
    g.check("workspace")
    gy.check("output")
    assert binding.last_device_status() == binding.PROM_OK
    assert np.array_equal(y.cpu().numpy(), want[-1])
    flags = []
    for i in range(seq.n - 1):
        off, chained = binding.debug_layer_seq_output_offset(seq, batch, h0, w0, i)
        flags.append(chained)
        if chained:
            got = ws[off:off + want[i].size].view(torch.int8).cpu().numpy().reshape(want[i].shape)
            assert first_mismatch(got.reshape(-1, got.shape[-1]), want[i].reshape(-1, got.shape[-1])) is None, i
    if expect_chained is not None:
        assert flags == expect_chained, flags
    return flags, want


def test_every_intermediate_of_the_network(oracle):
    """MobileNetV2's 34 layers at a reduced image size: the final output, the intermediates of
    the depth-first launches straight from the workspace, and every other intermediate as the
    result of the sequence cut short after that layer (prefixes also cut the runs short)."""
    table = synth.mobilenetv2_pointwise_layers(h0=64, w0=64)
    shapes = [(l.cin, l.cout, l.in_stride) for l in table]
    host, seq, dev = make_stack(51, shapes)
    x0 = synth.act_post_relu6(51, (3, 64, 64, 32))
    flags, want = run_and_check_all(oracle, host, seq, x0)
    assert sum(flags) >= 20, flags             # the late layers run depth-first
    for p in range(1, len(shapes)):
        sub = binding.LayerSeq(dev[:p])
        ws = torch.empty((max(16, sub.workspace_bytes(3, 64, 64)),), dtype=torch.uint8, device="cuda")
        y = binding.pw_layer_seq(sub, x0.cuda(), ws)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want[p - 1]), p
    assert binding.last_device_status() == binding.PROM_OK


def test_depth_first_and_layer_by_layer_agree(oracle):
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32)
    shapes = [(l.cin, l.cout, l.in_stride) for l in table]
    host, seq, _ = make_stack(52, shapes)
    x0 = synth.act_post_relu6(52, (5, 32, 32, 32)).cuda()
    ws = torch.empty((seq.workspace_bytes(5, 32, 32),), dtype=torch.uint8, device="cuda")
    y1 = binding.pw_layer_seq(seq, x0, ws).clone()
    try:
        binding.debug_seq_chain(0)
        assert not any(binding.debug_layer_seq_output_offset(seq, 5, 32, 32, i)[1] for i in range(seq.n - 1))
        y0 = binding.pw_layer_seq(seq, x0, ws).clone()
    finally:
        binding.debug_seq_chain(1)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)
    assert np.array_equal(y1.cpu().numpy(), oracle.layer_seq(host, x0.cpu().numpy()))


def test_several_tiles_per_cta_and_a_ragged_last_tile(oracle):
    """More tiles than resident CTAs (a CTA interleaves two or three of them), a number of rows
    that is not a multiple of the tile, layers with one and with several subtiles and K chunks."""
    shapes = [(32, 192, 1), (192, 32, 1), (32, 96, 1), (96, 160, 1), (160, 64, 1)]
    host, seq, _ = make_stack(53, shapes)
    x0 = synth.act_post_relu6(53, (1, 701, 127, 32))         # 89 027 rows: 696 tiles
    run_and_check_all(oracle, host, seq, x0, expect_chained=[True] * 4)


def test_run_that_starts_with_a_subsampled_input(oracle):
    """The first layer of a run reads every second pixel of every second line (a 3-D tensor
    map); tiles are then whole lines of the smaller image."""
    shapes = [(48, 32, 1), (32, 64, 2), (64, 320, 1), (320, 64, 1), (64, 1280, 1)]
    host, seq, _ = make_stack(54, shapes)
    x0 = synth.act_post_relu6(54, (7, 36, 28, 48))           # 14 x 18 output lines of 14 pixels
    flags, _ = run_and_check_all(oracle, host, seq, x0)
    assert flags == [False, True, True, True], flags


def test_run_with_a_layer_on_the_64_bit_epilogue(oracle):
    shapes = [(64, 96, 1), (96, 64, 1), (64, 128, 1)]
    host, seq, _ = make_stack(55, shapes, shift_span=1)
    x0 = synth.act_post_relu6(55, (2, 24, 20, 64))
    run_and_check_all(oracle, host, seq, x0, expect_chained=[True, True])


def test_layers_a_run_cannot_take_split_it(oracle):
    """Channel counts that are not multiples of 16 end a run; what is left on either side
    still runs depth-first when at least two layers remain."""
    shapes = [(32, 64, 1), (64, 96, 1), (96, 24, 1), (24, 64, 1), (64, 32, 1), (32, 64, 1), (64, 48, 1)]
    host, seq, _ = make_stack(56, shapes)
    x0 = synth.act_post_relu6(56, (2, 16, 16, 32))
    flags, _ = run_and_check_all(oracle, host, seq, x0)
    assert flags == [True, True, False, False, True, True], flags
