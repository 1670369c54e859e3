"""GPU parity of the layer sequence and of the benchmark configurations."""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding, build, synth
from gpu_util import first_mismatch, make_case, oracle_y, run_variant, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    build.build()
    binding.lib()
    binding.last_device_status()
    yield
    assert binding.last_device_status() == binding.PROM_OK


def build_sequence(seed, table, zero_frac=0.5):
    host, dev = [], []
    for i, l in enumerate(table):
        d = synth.make_layer(seed, l.cin, l.cout, zero_frac, index=i + 1)
        host.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w=d["w"].numpy(),
                         bias=d["bias"].numpy(), mult=d["mult"].numpy(), shift=d["shift"].numpy()))
        dev.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride,
                        w_packed=binding.pack_ternary(d["w"].cuda()), bias=d["bias"].cuda(),
                        mult=d["mult"].cuda(), shift=d["shift"].cuda()))
    return host, binding.LayerSeq(dev)


@pytest.mark.parametrize("variant", ["auto", "naive", "tc"])
@pytest.mark.parametrize("batch,hw", [(2, 32), (3, 64)])
def test_mobilenetv2_sequence_small(oracle, variant, batch, hw):
    """All 34 layers, chained, at a reduced image size (several tiles per layer
    early on, ragged tiles and single-tile layers late)."""
    table = synth.mobilenetv2_pointwise_layers(h0=hw, w0=hw)
    host, seq = build_sequence(31, table)
    x0 = synth.act_post_relu6(31, (batch, hw, hw, 32))
    ws = torch.empty((seq.workspace_bytes(batch, hw, hw),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq, x0.cuda(), ws, variant=variant)
    torch.cuda.synchronize()
    want = oracle.layer_seq(host, x0.numpy())
    assert y.shape == want.shape
    assert first_mismatch(y.cpu().numpy().reshape(-1, 1280), want.reshape(-1, 1280)) is None


@pytest.mark.parametrize("width", [0.75, 1.4, 2.0])
def test_mobilenetv2_sequence_width_multipliers(oracle, width):
    """The widths the paper sweeps (Section 5: 0.75x to 2.0x): channel counts such as
    72, 120, 136, 224, 448, 1344 and 2560, most of them not multiples of 32, some only of 8."""
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32, width=width)
    host, seq = build_sequence(33, table)
    x0 = synth.act_post_relu6(33, (2, 32, 32, table[0].cin))
    ws = torch.empty((seq.workspace_bytes(2, 32, 32),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq, x0.cuda(), ws)
    torch.cuda.synchronize()
    want = oracle.layer_seq(host, x0.numpy())
    assert y.shape == want.shape
    c = table[-1].cout
    assert first_mismatch(y.cpu().numpy().reshape(-1, c), want.reshape(-1, c)) is None
    assert binding.last_device_status() == binding.PROM_OK


@pytest.mark.parametrize("width", [0.75, 1.4])
def test_width_multiplier_layers_on_the_tensor_cores(oracle, width):
    """Every distinct (Cin, Cout) of a scaled network as a single tensor-core call with
    a ragged number of rows, where the tensor-core variant takes the shape."""
    seen = set()
    for l in synth.mobilenetv2_pointwise_layers(width=width):
        if (l.cin, l.cout) in seen:
            continue
        seen.add((l.cin, l.cout))
        m = 300
        x = synth.act_uniform_i8(34, (m, l.cin))
        lay = synth.make_layer(34, l.cin, l.cout, 0.5, index=len(seen))
        want = oracle.conv_mul(x.numpy(), lay["w"].numpy(), lay["bias"].numpy(),
                               lay["mult"].numpy(), lay["shift"].numpy())
        wp = binding.pack_ternary(lay["w"].cuda())
        rq = binding.make_requant(lay["bias"].cuda(), lay["mult"].cuda(), lay["shift"].cuda())
        for variant in ("auto", "tc"):
            try:
                y = binding.pw_conv_i8(x.cuda(), wp, l.cout, rq, variant=variant)
            except binding.PromError as e:
                assert variant == "tc" and e.code == binding.PROM_ERR_UNSUPPORTED, (l, variant, e)
                continue
            torch.cuda.synchronize()
            assert first_mismatch(y.cpu().numpy(), want) is None, (l.cin, l.cout, variant)


@pytest.mark.parametrize("batch,hw", [(2, 32), (1, 64)])
def test_sequence_with_real_depthwise_convolutions(oracle, batch, hw):
    """The body of the network with the int8 depthwise 3x3 in front of every project
    convolution (stride in the depthwise layer) instead of the identity stand-in, against the
    oracle's depthwise and pointwise functions applied layer by layer."""
    table = synth.mobilenetv2_pointwise_layers(h0=hw, w0=hw)
    rng = np.random.default_rng(35)
    host, dev = [], []
    for i, l in enumerate(table):
        d = synth.make_layer(35, l.cin, l.cout, 0.5, index=i + 1)
        hl = dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                  mult=d["mult"].numpy(), shift=d["shift"].numpy())
        dl = dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                  bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda())
        if l.name.endswith("project"):
            hl["dw_w"] = rng.integers(-20, 21, size=(l.cin, 3, 3)).astype(np.int8)
            hl["dw_bias"] = rng.integers(-64, 65, size=l.cin).astype(np.int32)
            hl["dw_mult"] = rng.integers(1 << 30, (1 << 31) - 1, size=l.cin).astype(np.int32)
            hl["dw_shift"] = rng.integers(5, 8, size=l.cin).astype(np.int8)
            for k in ("dw_w", "dw_bias", "dw_mult", "dw_shift"):
                dl[k] = torch.from_numpy(hl[k]).cuda()
        host.append(hl); dev.append(dl)
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(35, (batch, hw, hw, 32))
    ws = torch.empty((seq.workspace_bytes(batch, hw, hw),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq, x0.cuda(), ws)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    cur = x0.numpy()
    for hl in host:
        if "dw_w" in hl:
            cur = oracle.dw3x3(cur, hl["dw_w"], hl["dw_bias"], hl["dw_mult"], hl["dw_shift"],
                               stride=hl["in_stride"], act_min=0, act_max=127)
        elif hl["in_stride"] != 1:
            cur = oracle.subsample(cur, hl["in_stride"])
        b, h, w, c = cur.shape
        out = oracle.conv_mul(cur.reshape(-1, c), hl["w"], hl["bias"], hl["mult"], hl["shift"])
        cur = out.reshape(b, h, w, hl["cout"])
    assert y.shape == cur.shape
    assert first_mismatch(y.cpu().numpy().reshape(-1, 1280), cur.reshape(-1, 1280)) is None
    assert (cur != 0).mean() > 0.05          # the chain has not collapsed to zeros


def test_sequence_host_entry_point(oracle):
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32)[:9]
    host, seq = build_sequence(32, table)
    x0 = synth.act_post_relu6(32, (2, 32, 32, 32))
    ws = torch.empty((seq.host_workspace_bytes(2, 32, 32),), dtype=torch.uint8, device="cuda")
    want = oracle.layer_seq(host, x0.numpy())
    yh = torch.empty(want.shape, dtype=torch.int8).pin_memory()
    binding.pw_layer_seq_host(seq, x0.pin_memory(), ws, yh)
    torch.cuda.synchronize()
    assert np.array_equal(yh.numpy(), want)


def test_every_layer_standalone_at_its_channel_counts(oracle):
    """Each of the 34 layer shapes on a fresh seeded post-ReLU6 input (chained
    activations shrink towards the bias, which makes them weak evidence)."""
    table = synth.mobilenetv2_pointwise_layers()
    seen = set()
    for i, l in enumerate(table):
        if (l.cin, l.cout) in seen:
            continue
        seen.add((l.cin, l.cout))
        m = 1000 + 2 * i
        x, lay = make_case(100 + i, m, l.cin, l.cout, act="relu6")
        got = run_variant(*to_device(x, lay), l.cout, "auto")
        assert first_mismatch(got, oracle_y(oracle, x, lay)) is None, l


def test_config1_and_config4_shapes(oracle):
    for seed, (m, cin, cout, act) in enumerate([(196, 64, 384, "i8"), (3000, 960, 160, "u7"),
                                                (3000, 160, 960, "u7"), (3000, 320, 1280, "u7")]):
        x, lay = make_case(synth.BASE_SEED + seed, m, cin, cout, act=act)
        xd, wp, consts = to_device(x, lay)
        want = oracle_y(oracle, x, lay)
        for variant in ["tc", "addsub"]:
            got = run_variant(xd, wp, consts, cout, variant)
            assert first_mismatch(got, want) is None, (m, cin, cout, variant)


def test_config2_full_size_sampled_rows(oracle):
    """Config 2 at full size (M = 802816) in the launch shape the benchmark
    times; the oracle evaluates sampled rows (rows are independent)."""
    m, cin, cout = 64 * 112 * 112, 16, 96
    x = synth.act_post_relu6(synth.BASE_SEED + 2, (m, cin), device="cuda")
    lay = synth.make_layer(synth.BASE_SEED + 2, cin, cout, 0.5)
    wp = binding.pack_ternary(lay["w"].cuda())
    consts = (lay["bias"].cuda(), lay["mult"].cuda(), lay["shift"].cuda())
    rows = np.unique(np.concatenate([np.arange(0, 512), np.arange(m - 512, m),
                                     np.random.default_rng(0).integers(0, m, 20000)]))
    xs = x[torch.from_numpy(rows).cuda()].cpu()
    want = oracle_y(oracle, xs, lay)
    for variant in ["tc", "smallk", "auto"]:
        y = torch.empty((m, cout), dtype=torch.int8, device="cuda")
        binding.pw_conv_i8(x, wp, cout, binding.make_requant(*consts), y=y, variant=variant)
        got = y[torch.from_numpy(rows).cuda()].cpu().numpy()
        assert first_mismatch(got, want) is None, variant
        # all variants agree everywhere
        if variant == "tc":
            ref = y.clone()
        else:
            assert torch.equal(y, ref)


def test_every_layer_shape_many_tiles_per_cta(oracle):
    """Each MobileNetV2 layer shape at a row count that gives every CTA several
    tiles, so that the rings of activation stages and accumulators wrap many
    times: the tensor-core variant against the one-thread-per-output kernel on
    the whole tensor, and against the oracle on sampled rows."""
    table = synth.mobilenetv2_pointwise_layers()
    seen = set()
    m = 128 * 148 * 4 + 78
    rows = np.unique(np.concatenate([np.arange(0, 300), np.arange(m - 300, m),
                                     np.random.default_rng(1).integers(0, m, 1500)]))
    for i, l in enumerate(table):
        if (l.cin, l.cout) in seen:
            continue
        seen.add((l.cin, l.cout))
        x = synth.act_post_relu6(200 + i, (m, l.cin), device="cuda")
        lay = synth.make_layer(200 + i, l.cin, l.cout, 0.5)
        wp = binding.pack_ternary(lay["w"].cuda())
        rq = binding.make_requant(lay["bias"].cuda(), lay["mult"].cuda(), lay["shift"].cuda())
        y_tc = torch.full((m, l.cout), -3, dtype=torch.int8, device="cuda")
        y_nv = torch.full((m, l.cout), -4, dtype=torch.int8, device="cuda")
        binding.pw_conv_i8(x, wp, l.cout, rq, y=y_tc, variant="tc")
        binding.pw_conv_i8(x, wp, l.cout, rq, y=y_nv, variant="naive")
        torch.cuda.synchronize()
        assert binding.last_device_status() == binding.PROM_OK, l
        assert torch.equal(y_tc, y_nv), l
        idx = torch.from_numpy(rows).cuda()
        want = oracle_y(oracle, x[idx].cpu(), lay)
        assert first_mismatch(y_tc[idx].cpu().numpy(), want) is None, l


def test_config3_full_size_sequence(oracle):
    """The benchmark's own launch: all 34 layers at batch 128.  The library's
    choice of variants against the plain kernel on the whole output, and the
    oracle on the first two images (images are independent)."""
    table = synth.mobilenetv2_pointwise_layers()
    host, seq = build_sequence(synth.BASE_SEED + 3, table)
    x0 = synth.act_post_relu6(synth.BASE_SEED + 3, (128, 112, 112, 32), device="cuda")
    ws = torch.empty((seq.workspace_bytes(128, 112, 112),), dtype=torch.uint8, device="cuda")
    y_auto = binding.pw_layer_seq(seq, x0, ws, variant="auto").clone()
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    y_naive = binding.pw_layer_seq(seq, x0, ws, variant="naive")
    torch.cuda.synchronize()
    assert torch.equal(y_auto, y_naive)
    want = oracle.layer_seq(host, x0[:2].cpu().numpy())
    assert np.array_equal(y_auto[:2].cpu().numpy(), want)


def test_sequence_with_small_workspace_and_mixed_variants(oracle):
    """The prepared-operand images are an optimisation: a workspace that only
    holds the two activation regions gives the same bytes.  The second half
    mixes in layers the tensor-core variant refuses (Cin = 20, Cout = 12), which
    AUTO runs on other kernels inside the same chained call."""
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32)[:12]
    host, seq = build_sequence(41, table)
    x0 = synth.act_post_relu6(41, (4, 32, 32, 32))
    want = oracle.layer_seq(host, x0.numpy())
    full = seq.workspace_bytes(4, 32, 32)
    regions = 0
    h = w = 32
    sizes = []
    for l in table:
        h //= l.in_stride; w //= l.in_stride
        sizes.append((4 * h * w * l.cout + 255) // 256 * 256)
    regions = max(sizes[0:-1:2]) + max(sizes[1:-1:2])
    assert regions < full
    for nbytes in (full, regions):
        ws = torch.empty((nbytes,), dtype=torch.uint8, device="cuda")
        y = binding.pw_layer_seq(seq, x0.cuda(), ws)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want), nbytes

    shapes = [(32, 64, 1), (64, 20, 1), (20, 12, 1), (12, 48, 2), (48, 16, 1)]
    host, dev = [], []
    for i, (cin, cout, stride) in enumerate(shapes):
        d = synth.make_layer(42, cin, cout, 0.5, index=i + 1)
        host.append(dict(cin=cin, cout=cout, in_stride=stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                         mult=d["mult"].numpy(), shift=d["shift"].numpy()))
        dev.append(dict(cin=cin, cout=cout, in_stride=stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                        bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda()))
    seq2 = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(42, (3, 16, 16, 32))
    ws = torch.empty((max(16, seq2.workspace_bytes(3, 16, 16)),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq2, x0.cuda(), ws, variant="auto")
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), oracle.layer_seq(host, x0.numpy()))
    with pytest.raises(binding.PromError) as e:
        binding.pw_layer_seq(seq2, x0.cuda(), ws, variant="tc")
    assert e.value.code == binding.PROM_ERR_UNSUPPORTED


def test_sequence_twice_and_in_a_cuda_graph(oracle):
    """Two calls in a row reuse the workspace (the images are rebuilt each time),
    and a captured call replays to the same bytes."""
    table = synth.mobilenetv2_pointwise_layers(h0=32, w0=32)
    host, seq = build_sequence(43, table)
    x0 = synth.act_post_relu6(43, (2, 32, 32, 32)).cuda()
    want = oracle.layer_seq(host, x0.cpu().numpy())
    ws = torch.empty((seq.workspace_bytes(2, 32, 32),), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    y = torch.zeros(want.shape, dtype=torch.int8, device="cuda")
    with torch.cuda.stream(side):
        for _ in range(2):
            binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), want)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        binding.pw_layer_seq(seq, x0, ws, y_out=y, stream=side)
    for _ in range(3):
        y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), want)
    assert binding.last_device_status() == binding.PROM_OK


def test_seeded_random_stacks(oracle):
    """Twelve seeded random stacks of 2-6 layers: random channel counts (multiples of 8),
    strides, image sizes, and a depthwise 3x3 in front of some layers, against the oracle's
    functions applied layer by layer."""
    rng = np.random.default_rng(777)
    for case in range(12):
        n = int(rng.integers(2, 7))
        batch = int(rng.integers(1, 4))
        h = int(rng.choice([8, 12, 16, 24])); w = int(rng.choice([8, 12, 16, 20]))
        chans = [8 * int(rng.integers(1, 41)) for _ in range(n + 1)]
        host, dev = [], []
        hh, ww = h, w
        for i in range(n):
            stride = 2 if (hh % 2 == 0 and ww % 2 == 0 and hh >= 4 and ww >= 4 and rng.random() < 0.35) else 1
            hh //= stride; ww //= stride
            d = synth.make_layer(500 + case, chans[i], chans[i + 1], 0.5, index=i + 1)
            hl = dict(cin=chans[i], cout=chans[i + 1], in_stride=stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                      mult=d["mult"].numpy(), shift=d["shift"].numpy())
            dl = dict(cin=chans[i], cout=chans[i + 1], in_stride=stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                      bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda())
            if rng.random() < 0.4:
                c = chans[i]
                hl["dw_w"] = rng.integers(-30, 31, size=(c, 3, 3)).astype(np.int8)
                hl["dw_bias"] = rng.integers(-64, 65, size=c).astype(np.int32)
                hl["dw_mult"] = rng.integers(1 << 30, (1 << 31) - 1, size=c).astype(np.int32)
                hl["dw_shift"] = rng.integers(5, 8, size=c).astype(np.int8)
                for k in ("dw_w", "dw_bias", "dw_mult", "dw_shift"):
                    dl[k] = torch.from_numpy(hl[k]).cuda()
            host.append(hl); dev.append(dl)
        seq = binding.LayerSeq(dev)
        x0 = synth.act_post_relu6(500 + case, (batch, h, w, chans[0]))
        ws = torch.empty((max(seq.workspace_bytes(batch, h, w), 16),), dtype=torch.uint8, device="cuda")
        y = binding.pw_layer_seq(seq, x0.cuda(), ws)
        torch.cuda.synchronize()
        assert binding.last_device_status() == binding.PROM_OK, case
        cur = x0.numpy()
        for hl in host:
            if "dw_w" in hl:
                cur = oracle.dw3x3(cur, hl["dw_w"], hl["dw_bias"], hl["dw_mult"], hl["dw_shift"],
                                   stride=hl["in_stride"], act_min=0, act_max=127)
            elif hl["in_stride"] != 1:
                cur = oracle.subsample(cur, hl["in_stride"])
            b, ch_h, ch_w, c = cur.shape
            cur = oracle.conv_mul(cur.reshape(-1, c), hl["w"], hl["bias"], hl["mult"], hl["shift"]).reshape(
                b, ch_h, ch_w, hl["cout"])
        got = y.cpu().numpy()
        assert got.shape == cur.shape, (case, got.shape, cur.shape)
        assert np.array_equal(got, cur), (case, [(l["cin"], l["cout"], l["in_stride"], "dw_w" in l) for l in host])


def test_tile_order_does_not_change_the_bytes(oracle):
    """Every second layer walks its row tiles backwards by default: the same bytes as with every
    layer walking forwards, on a network with subsampled layers and ragged last tiles."""
    table = synth.mobilenetv2_pointwise_layers(h0=48, w0=80)
    host, dev = [], []
    for i, l in enumerate(table):
        d = synth.make_layer(91, l.cin, l.cout, 0.5, index=i + 1)
        host.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                         mult=d["mult"].numpy(), shift=d["shift"].numpy()))
        dev.append(dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                        bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda()))
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(91, (7, 48, 80, 32))
    ws = torch.empty((seq.workspace_bytes(7, 48, 80),), dtype=torch.uint8, device="cuda")
    y1 = binding.pw_layer_seq(seq, x0.cuda(), ws).clone()
    try:
        binding.debug_seq_order(False)
        y0 = binding.pw_layer_seq(seq, x0.cuda(), ws).clone()
    finally:
        binding.debug_seq_order(True)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    assert torch.equal(y0, y1)
    assert np.array_equal(y1.cpu().numpy(), oracle.layer_seq(host, x0.numpy()))
