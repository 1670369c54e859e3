"""GPU parity of the runs of layers that stay in shared memory inside a layer sequence.

With `prom_debug_seq_chain(2)` a run of consecutive layers on the same pixels (alternately
narrowing to at most 384 channels and widening again, as the blocks of the network do) is one
launch in which a CTA takes a tile of rows through every layer of the run, the activations never
leaving shared memory; only the run's last layer writes a tensor.  Every such output, and the output of
the sequence, is compared with the CPU oracle byte for byte, inside guarded buffers.
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
    binding.debug_seq_chain(2)
    yield
    binding.debug_seq_chain(0)
    assert binding.last_device_status() == binding.PROM_OK


def make_layers(seed, shapes, wide_shifts=(), clamps=None):
    """shapes: [(cin, cout, in_stride)]; wide_shifts: layers whose shifts span more than 4 (the
    64-bit epilogue); clamps: {layer: (lo, hi)}."""
    host, dev = [], []
    clamps = clamps or {}
    for i, (cin, cout, stride) in enumerate(shapes):
        d = synth.make_layer(seed, cin, cout, 0.5, index=i + 1)
        if i in wide_shifts:
            d["shift"][: max(1, cout // 3)] = 1
        lo, hi = clamps.get(i, (0, 127))
        host.append(dict(cin=cin, cout=cout, in_stride=stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                         mult=d["mult"].numpy(), shift=d["shift"].numpy(), lo=lo, hi=hi))
        dev.append(dict(cin=cin, cout=cout, in_stride=stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                        bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda(),
                        act_min=lo, act_max=hi))
    return host, dev


def oracle_outputs(oracle, host, x0):
    outs, cur = [], x0
    for hl in host:
        if hl["in_stride"] != 1:
            cur = oracle.subsample(cur, hl["in_stride"])
        b, h, w, c = cur.shape
        cur = oracle.conv_mul(cur.reshape(-1, c), hl["w"], hl["bias"], hl["mult"], hl["shift"], hl["lo"],
                              hl["hi"]).reshape(b, h, w, hl["cout"])
        outs.append(cur)
    return outs


def run_and_check(oracle, host, dev, x0, expect=None):
    """Runs the sequence in guarded buffers; compares its output and every tensor that a run wrote
    to the workspace.  Returns per layer 'inner' (no tensor), 'last' (of a run) or 'plain'."""
    seq = binding.LayerSeq(dev)
    batch, h0, w0, _ = x0.shape
    want = oracle_outputs(oracle, host, x0.numpy())
    nbytes = max(16, seq.workspace_bytes(batch, h0, w0))
    g = Guarded(nbytes, dtype=torch.uint8, fill=0xEE)
    ws = g.view(nbytes)
    gy = Guarded(want[-1].size)
    y = gy.view(*want[-1].shape)
    binding.pw_layer_seq(seq, x0.cuda(), ws, y_out=y)
    torch.cuda.synchronize()
    g.check("workspace")
    gy.check("output")
    assert binding.last_device_status() == binding.PROM_OK
    got = y.cpu().numpy()
    assert first_mismatch(got.reshape(-1, got.shape[-1]), want[-1].reshape(-1, got.shape[-1])) is None
    kinds = []
    for i in range(seq.n - 1):
        off, chained = binding.debug_layer_seq_output_offset(seq, batch, h0, w0, i)
        kinds.append("inner" if off == -2 else ("last" if chained else "plain"))
        if off >= 0 and chained:        # (the ping-pong regions of the other layers are reused)
            t = ws[off:off + want[i].size].view(torch.int8).cpu().numpy().reshape(want[i].shape)
            assert first_mismatch(t.reshape(-1, t.shape[-1]), want[i].reshape(-1, t.shape[-1])) is None, i
    if expect is not None:
        assert kinds == expect, kinds
    return kinds, want


def test_one_run_several_tiles_ragged_end(oracle):
    """Eighteen row tiles, the last one short; one and several column tiles and K chunks."""
    shapes = [(192, 64, 1), (64, 384, 1), (384, 64, 1), (64, 384, 1), (384, 96, 1), (96, 576, 1)]
    host, dev = make_layers(61, shapes)
    x0 = synth.act_post_relu6(61, (1, 57, 40, 192))
    run_and_check(oracle, host, dev, x0, expect=["inner"] * 5)


def test_more_tiles_than_sms(oracle):
    """Several tiles per CTA: the input buffer, the rings and every barrier go round."""
    shapes = [(144, 32, 1), (32, 192, 1), (192, 32, 1), (32, 96, 1), (96, 160, 1), (160, 64, 1)]
    host, dev = make_layers(62, shapes)
    x0 = synth.act_post_relu6(62, (1, 701, 127, 144))        # 89 027 rows: 696 tiles
    run_and_check(oracle, host, dev, x0, expect=["inner"] * 5)


def test_subsampled_input_wide_layers_and_a_following_layer(oracle):
    """A run that starts with every second pixel of every second line (tiles are whole lines of the
    smaller image), widths up to 960 and a layer with three live accumulators (960 -> 320), then a
    layer outside the run that reads the run's output from the workspace."""
    shapes = [(48, 576, 1), (576, 160, 2), (160, 960, 1), (960, 160, 1), (160, 960, 1), (960, 320, 1),
              (320, 1280, 1), (1280, 24, 1)]
    host, dev = make_layers(63, shapes)
    x0 = synth.act_post_relu6(63, (5, 28, 28, 48))
    kinds, _ = run_and_check(oracle, host, dev, x0)
    assert kinds[1:6] == ["inner"] * 5 and kinds[6] == "last", kinds


def test_both_epilogues_and_clamps(oracle):
    """Layers on the 64-bit epilogue (wide shift spans, a signed clamp, a narrow clamp) between
    layers on the one-multiply form; signed activations flow into the next layer."""
    shapes = [(128, 256, 1), (256, 48, 1), (48, 272, 1), (272, 80, 1), (80, 144, 1)]
    host, dev = make_layers(64, shapes, wide_shifts=(1, 3), clamps={0: (-128, 127), 2: (-7, 99), 4: (-128, 127)})
    x0 = synth.act_post_relu6(64, (2, 33, 31, 128))
    run_and_check(oracle, host, dev, x0, expect=["inner"] * 4)


def test_the_network_and_its_prefixes(oracle):
    """MobileNetV2's 34 layers at a reduced image size, and the sequence cut short after every
    layer (which cuts the runs short too): each prefix's output against the oracle."""
    table = synth.mobilenetv2_pointwise_layers(h0=64, w0=64)
    shapes = [(l.cin, l.cout, l.in_stride) for l in table]
    host, dev = make_layers(65, shapes)
    x0 = synth.act_post_relu6(65, (3, 64, 64, 32))
    kinds, want = run_and_check(oracle, host, dev, x0)
    assert kinds.count("inner") >= 15, kinds
    for p in range(1, len(shapes)):
        sub = binding.LayerSeq(dev[:p])
        ws = torch.empty((max(16, sub.workspace_bytes(3, 64, 64)),), dtype=torch.uint8, device="cuda")
        y = binding.pw_layer_seq(sub, x0.cuda(), ws)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want[p - 1]), p
    assert binding.last_device_status() == binding.PROM_OK


def test_same_bytes_as_one_launch_per_layer():
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32)
    shapes = [(l.cin, l.cout, l.in_stride) for l in table]
    _, dev = make_layers(66, shapes)
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(66, (9, 32, 32, 32)).cuda()
    ws = torch.empty((seq.workspace_bytes(9, 32, 32),), dtype=torch.uint8, device="cuda")
    y1 = binding.pw_layer_seq(seq, x0, ws).clone()
    try:
        binding.debug_seq_chain(0)
        ws0 = torch.empty((seq.workspace_bytes(9, 32, 32),), dtype=torch.uint8, device="cuda")
        y0 = binding.pw_layer_seq(seq, x0, ws0).clone()
    finally:
        binding.debug_seq_chain(2)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)
