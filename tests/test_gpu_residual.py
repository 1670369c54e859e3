"""Parity of the project convolution with its skip connection (prom_pw_conv_i8_res and the
add_block_input flag of a layer sequence) against the oracle: the layer, then the clamped int8
sum with the block's input."""
import numpy as np
import pytest
import torch

from gpu_util import first_mismatch, make_case, oracle_y, to_device
from paper_2505_03254_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _residual(seed, m, cout):
    # values that reach both ends of the int8 range, so that sums saturate on both sides
    g = torch.Generator().manual_seed(seed + 17)
    return torch.randint(-128, 128, (m, cout), generator=g, dtype=torch.int32).to(torch.int8)


def _run(xd, wp, consts, cout, res_d, variant, act_min, act_max, in_place=False):
    rq = binding.make_requant(*consts, act_min, act_max)
    if in_place:
        y = res_d.clone()
        binding.pw_conv_i8_res(xd, wp, cout, rq, y, y=y, variant=variant)
    else:
        y = torch.full((xd.shape[0], cout), -77, dtype=torch.int8, device="cuda")
        binding.pw_conv_i8_res(xd, wp, cout, rq, res_d, y=y, variant=variant)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    return y.cpu().numpy()


# shapes: the project layers of the network's skip blocks (rows of a small image), ragged row
# counts, one subtile and several, 8-modulo-16 widths (folded rows), a wide output
SHAPES = [(3136, 144, 24), (784, 192, 32), (1000, 384, 64), (777, 576, 96), (98, 960, 160),
          (4096, 96, 24), (130, 64, 8), (2, 32, 16), (5000, 32, 320), (1234, 128, 136),
          (33, 48, 40), (6272, 16, 96)]


@pytest.mark.parametrize("m,cin,cout", SHAPES)
@pytest.mark.parametrize("clamp", [(-128, 127), (0, 127), (-20, 90)])
def test_layer_plus_residual_matches_the_oracle(oracle, m, cin, cout, clamp):
    x, lay = make_case(1100 + cin + cout, m, cin, cout)
    res = _residual(m + cout, m, cout)
    want = oracle.residual_add(oracle_y(oracle, x, lay, *clamp), res.numpy())
    xd, wp, consts = to_device(x, lay)
    res_d = res.cuda()
    for variant in ("auto", "tc", "naive"):
        try:
            got = _run(xd, wp, consts, cout, res_d, variant, *clamp)
        except binding.PromError as e:
            # odd row counts with widths that are not multiples of 16 are outside the tensor-core route
            assert variant == "tc" and e.code == binding.PROM_ERR_UNSUPPORTED and (m & 1), (variant, e)
            continue
        assert first_mismatch(got, want) is None, variant
    # the sum formed in place over the residual
    got = _run(xd, wp, consts, cout, res_d, "auto", *clamp, in_place=True)
    assert first_mismatch(got, want) is None
    if m >= 500 and clamp[0] < 0:
        assert (want == 127).any() and (want == -128).any()  # sums saturated on both sides


def test_variants_without_a_fused_sum_refuse(oracle):
    x, lay = make_case(5, 64, 32, 16)
    xd, wp, consts = to_device(x, lay)
    rq = binding.make_requant(*consts, 0, 127)
    res = _residual(1, 64, 16).cuda()
    for variant in ("smallk", "addsub"):
        with pytest.raises(binding.PromError) as e:
            binding.pw_conv_i8_res(xd, wp, 16, rq, res, variant=variant)
        assert e.value.code == binding.PROM_ERR_UNSUPPORTED
    with pytest.raises(ValueError):
        binding.pw_conv_i8_res(xd, wp, 16, rq, res[:32])
    # an empty matrix is a no-op
    empty = torch.empty((0, 32), dtype=torch.int8, device="cuda")
    out = binding.pw_conv_i8_res(empty, wp, 16, rq, torch.empty((0, 16), dtype=torch.int8, device="cuda"))
    assert out.shape == (0, 16)


def test_full_size_layer_sampled_rows(oracle):
    """A project layer of the network at batch 128 (56x56 images, 144 -> 24 channels): sampled
    rows against the oracle, in place over the residual."""
    m, cin, cout = 128 * 56 * 56, 144, 24
    x = synth.act_post_relu6(77, (m, cin), device="cuda")
    lay = synth.make_layer(77, cin, cout, 0.5)
    g = torch.Generator(device="cuda").manual_seed(3)
    res = torch.randint(-128, 128, (m, cout), generator=g, dtype=torch.int32, device="cuda").to(torch.int8)
    rq = binding.make_requant(lay["bias"].cuda(), lay["mult"].cuda(), lay["shift"].cuda(), -128, 127)
    y = res.clone()
    binding.pw_conv_i8_res(x, binding.pack_ternary(lay["w"].cuda()), cout, rq, y, y=y)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    idx = torch.cat([torch.arange(0, 300), torch.randint(0, m, (3000,), generator=torch.Generator().manual_seed(1)),
                     torch.arange(m - 300, m)])
    want = oracle.residual_add(oracle_y(oracle, x[idx.cuda()].cpu(), lay, -128, 127), res[idx.cuda()].cpu().numpy())
    assert first_mismatch(y[idx.cuda()].cpu().numpy(), want) is None


def _body(seed, hw, with_depthwise):
    """The network's pointwise layers with linear project layers and the skip connections of
    its ten shape-preserving blocks; host and device descriptions."""
    table = synth.mobilenetv2_pointwise_layers(h0=hw, w0=hw)
    rng = np.random.default_rng(seed)
    host, dev = [], []
    for i, l in enumerate(table):
        d = synth.make_layer(seed, l.cin, l.cout, 0.5, index=i + 1)
        linear = l.name.endswith("project")
        hl = dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w=d["w"].numpy(), bias=d["bias"].numpy(),
                  mult=d["mult"].numpy(), shift=d["shift"].numpy(), act_min=-128 if linear else 0,
                  skip=synth.has_skip_connection(table, i))
        dl = dict(cin=l.cin, cout=l.cout, in_stride=l.in_stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                  bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda(),
                  act_min=hl["act_min"], add_block_input=hl["skip"])
        if with_depthwise and linear:
            hl["dw_w"] = rng.integers(-20, 21, size=(l.cin, 3, 3)).astype(np.int8)
            hl["dw_bias"] = rng.integers(-64, 65, size=l.cin).astype(np.int32)
            hl["dw_mult"] = rng.integers(1 << 30, (1 << 31) - 1, size=l.cin).astype(np.int32)
            hl["dw_shift"] = rng.integers(5, 8, size=l.cin).astype(np.int8)
            for k in ("dw_w", "dw_bias", "dw_mult", "dw_shift"):
                dl[k] = torch.from_numpy(hl[k]).cuda()
        host.append(hl); dev.append(dl)
    return host, dev


def _oracle_body(oracle, host, x0):
    cur, inputs = x0, []
    for hl in host:
        inputs.append(cur)
        if "dw_w" in hl:
            cur = oracle.dw3x3(cur, hl["dw_w"], hl["dw_bias"], hl["dw_mult"], hl["dw_shift"],
                               stride=hl["in_stride"], act_min=0, act_max=127)
        elif hl["in_stride"] != 1:
            cur = oracle.subsample(cur, hl["in_stride"])
        b, h, w, c = cur.shape
        out = oracle.conv_mul(cur.reshape(-1, c), hl["w"], hl["bias"], hl["mult"], hl["shift"],
                              hl["act_min"], 127).reshape(b, h, w, hl["cout"])
        if hl["skip"]:
            out = oracle.residual_add(out, inputs[-2])       # the input of the expand layer
        cur = out
    return cur


@pytest.mark.parametrize("with_depthwise", [False, True])
@pytest.mark.parametrize("variant", ["auto", "naive"])
@pytest.mark.parametrize("n_skips", [2, 10])
def test_network_body_with_skip_connections(oracle, with_depthwise, variant, n_skips):
    """The whole body (ten skip connections, then the head), and the body cut after its
    second skip connection, where the sum is the sequence's output."""
    host, dev = _body(61, 32, with_depthwise)
    assert sum(h["skip"] for h in host) == 10
    if n_skips < 10:
        cut = [i for i, h in enumerate(host) if h["skip"]][n_skips - 1] + 1
        host, dev = host[:cut], dev[:cut]
    seq = binding.LayerSeq(dev)
    x0 = synth.act_post_relu6(61, (2, 32, 32, 32))
    ws = torch.empty((seq.workspace_bytes(2, 32, 32),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq, x0.cuda(), ws, variant=variant)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    want = _oracle_body(oracle, host, x0.numpy())
    assert y.shape == want.shape
    c = want.shape[-1]
    assert first_mismatch(y.cpu().numpy().reshape(-1, c), want.reshape(-1, c)) is None
    assert (want != 0).mean() > 0.05
    if n_skips < 10:
        # the skip connections matter: without them the result differs
        for h in host:
            h["skip"] = False
        assert not np.array_equal(_oracle_body(oracle, host, x0.numpy()), want)


def test_skip_connection_from_the_sequence_input(oracle):
    """A block at the very start: the residual is the caller's input tensor, and the last
    layer of a sequence writes the sum to the caller's output."""
    layers = [(24, 144, 1), (144, 24, 1)]
    host, dev = [], []
    for i, (cin, cout, s) in enumerate(layers):
        d = synth.make_layer(9, cin, cout, 0.5, index=i + 1)
        host.append(dict(cin=cin, cout=cout, in_stride=s, w=d["w"].numpy(), bias=d["bias"].numpy(),
                         mult=d["mult"].numpy(), shift=d["shift"].numpy(), act_min=-128 if i else 0, skip=i == 1))
        dev.append(dict(cin=cin, cout=cout, in_stride=s, w_packed=binding.pack_ternary(d["w"].cuda()),
                        bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda(),
                        act_min=-128 if i else 0, add_block_input=i == 1))
    seq = binding.LayerSeq(dev)
    x0 = synth.act_uniform_i8(9, (3, 10, 14, 24))
    ws = torch.empty((seq.workspace_bytes(3, 10, 14),), dtype=torch.uint8, device="cuda")
    y = binding.pw_layer_seq(seq, x0.cuda(), ws)
    torch.cuda.synchronize()
    want = _oracle_body(oracle, host, x0.numpy())
    assert first_mismatch(y.cpu().numpy().reshape(-1, 24), want.reshape(-1, 24)) is None


def test_sequence_rejects_a_skip_that_does_not_fit(oracle):
    d0 = synth.make_layer(1, 16, 96, 0.5, index=1)
    d1 = synth.make_layer(1, 96, 24, 0.5, index=2)

    def dev(d, cin, cout, stride, flag):
        return dict(cin=cin, cout=cout, in_stride=stride, w_packed=binding.pack_ternary(d["w"].cuda()),
                    bias=d["bias"].cuda(), mult=d["mult"].cuda(), shift=d["shift"].cuda(), add_block_input=flag)

    x0 = synth.act_uniform_i8(1, (1, 8, 8, 16)).cuda()
    ws = torch.empty((1 << 20,), dtype=torch.uint8, device="cuda")
    # channel counts differ; a flag on the first layer; a stride inside the block
    for layers in ([dev(d0, 16, 96, 1, False), dev(d1, 96, 24, 1, True)],
                   [dev(d0, 16, 96, 1, True)],
                   [dev(d0, 16, 96, 1, False), dev(synth.make_layer(1, 96, 16, 0.5, index=2), 96, 16, 2, True)]):
        with pytest.raises(binding.PromError) as e:
            binding.pw_layer_seq(binding.LayerSeq(layers), x0, ws)
        assert e.value.code == binding.PROM_ERR_SHAPE
    # variants without a fused sum refuse the sequence
    ok = [dev(d0, 16, 96, 1, False), dev(synth.make_layer(1, 96, 16, 0.5, index=2), 96, 16, 1, True)]
    with pytest.raises(binding.PromError) as e:
        binding.pw_layer_seq(binding.LayerSeq(ok), x0, ws, variant="addsub")
    assert e.value.code == binding.PROM_ERR_UNSUPPORTED
