"""The seeded generators and workload tables, against independent statements."""
import os

import numpy as np
import torch

from paper_2505_03254_b200 import synth

M64 = (1 << 64) - 1


def py_hash(seed, stream, i):
    """SplitMix64 output function on Python integers (independent of torch)."""
    z = (seed + 0x9E3779B97F4A7C15 * (i + 1) + 0xD1B54A32D192ED03 * stream) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def test_hash_matches_python_integers():
    for seed, stream, start in [(0, 1, 0), (synth.BASE_SEED + 3, 2, 12345), (7, 5003, 1 << 33)]:
        got = synth.hash64(seed, stream, start, 16).tolist()
        want = [py_hash(seed, stream, start + i) for i in range(16)]
        assert [g & M64 for g in got] == want


def test_splitmix_known_vector():
    # SplitMix64 seeded with 0: the first outputs of the published generator.
    # state_n = n*GOLDEN, output = mix(state_n); our h(0, 0, i) is output i.
    want = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert [py_hash(0, 0, i) for i in range(3)] == want
    assert [v & M64 for v in synth.hash64(0, 0, 0, 3).tolist()] == want


def test_value_maps():
    seed = 11
    n = 4096
    hs = [py_hash(seed, synth.STREAM_X, i) for i in range(n)]
    x = synth.act_uniform_i8(seed, (n,)).tolist()
    assert x == [((h & 0xFF) ^ 0x80) - 0x80 for h in hs]
    x = synth.act_post_relu6(seed, (n,)).tolist()
    thr = int(0.3 * 2 ** 32)
    assert x == [0 if (h >> 32) < thr else (h & 0x7F) for h in hs]
    hw = [py_hash(seed, synth.STREAM_W, i) for i in range(n)]
    w = synth.ternary_weights(seed, 64, 64, 0.5).flatten().tolist()
    thr = int(0.5 * 2 ** 32)
    assert w == [0 if (h >> 32) < thr else (1 if h & 1 else -1) for h in hw]
    b, m, s = synth.requant_constants(seed, 200)
    hb = [py_hash(seed, synth.STREAM_BIAS, i) for i in range(200)]
    hm = [py_hash(seed, synth.STREAM_MULT, i) for i in range(200)]
    hh = [py_hash(seed, synth.STREAM_SHIFT, i) for i in range(200)]
    assert b.tolist() == [(h >> 11) % 8193 - 4096 for h in hb]
    assert m.tolist() == [(1 << 30) + (h & ((1 << 30) - 1)) for h in hm]
    assert s.tolist() == [8 + (h >> 40) % 5 for h in hh]


def test_distributions():
    n = 1 << 20
    for z in (0.3, 0.5, 0.7, 0.9):
        w = synth.ternary_weights(5, 1024, 1024, z)
        f0 = (w == 0).float().mean().item()
        sd = (z * (1 - z) / n) ** 0.5
        assert abs(f0 - z) < 5 * sd
        fp = (w == 1).float().mean().item()
        fm = (w == -1).float().mean().item()
        assert abs(fp - fm) < 5 * (1.0 / n) ** 0.5
    x = synth.act_post_relu6(5, (n,))
    assert x.min().item() == 0 and x.max().item() == 127
    f0 = (x == 0).float().mean().item()
    assert abs(f0 - (0.3 + 0.7 / 128)) < 0.003
    x = synth.act_uniform_i8(5, (n,))
    assert x.min().item() == -128 and x.max().item() == 127
    assert abs(x.float().mean().item() + 0.5) < 0.5
    b, m, s = synth.requant_constants(5, 100000)
    assert b.min().item() >= -4096 and b.max().item() <= 4096
    assert m.min().item() >= 1 << 30 and m.max().item() < 1 << 31
    assert set(s.tolist()) == {8, 9, 10, 11, 12}


def test_chunked_fill_is_index_addressed():
    # an element does not depend on how the tensor was chunked or shaped
    a = synth.act_uniform_i8(3, (1000, 7))
    b = synth.act_uniform_i8(3, (7000,))
    assert torch.equal(a.flatten(), b)


def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_cost_shares.txt")
    out = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            out[k.strip()] = float(v)
    return out


def test_layer_table_against_paper_figures():
    """The 34-layer table reproduces the parameter shares and the storage
    sizes the paper prints (Section 2; Table 1)."""
    g = _golden()
    layers = synth.mobilenetv2_pointwise_layers()
    assert len(layers) == 34
    assert (layers[0].cin, layers[0].cout) == (32, 16)
    assert (layers[-1].cin, layers[-1].cout, layers[-1].h) == (320, 1280, 7)
    assert sum(1 for l in layers if l.in_stride == 2) == 4
    pw = sum(l.cin * l.cout for l in layers)
    # the rest of MobileNetV2, from the same (t, c, n, s) table
    dw, bn = 0, 32
    c = 32
    for t, cout, n, s in synth.MOBILENETV2_TCNS:
        for r in range(n):
            hidden = c * t
            dw += 9 * hidden
            bn += (hidden if t != 1 else 0) + hidden + cout
            c = cout
    bn += 1280
    stem = 3 * 3 * 3 * 32
    linear = 1280 * 1000 + 1000
    no_bn = pw + dw + stem + linear
    assert abs(pw / no_bn - g["pointwise_param_share"]) < 0.0006
    assert abs(dw / no_bn - g["depthwise_param_share"]) < 0.0006
    total = no_bn + 2 * bn
    assert abs(total * 2 / 1e6 - g["fp16_size_mb_1_0x"]) < 0.006
    # ternary at 2 bits, everything else int8, BatchNorm kept in fp16
    prom_mb = (pw * 2 / 8 + (no_bn - pw) + 2 * bn * 2) / 1e6
    assert abs(prom_mb - g["prom_size_mb_1_0x"]) < 0.006
    # MACs per image: chaining and spatial sizes
    macs = sum(l.h * l.w * l.cin * l.cout for l in layers)
    assert macs == 267939840
    for a, b in zip(layers, layers[1:]):
        assert a.cout == b.cin
        assert b.h * b.in_stride == a.h


def test_width_multiplier_tables():
    """Width 1.0 is the plain table; scaled tables keep the block structure, channel counts
    stay multiples of 8 and within a tenth of the scaled value, the head grows only above 1.0."""
    base = synth.mobilenetv2_pointwise_layers()
    assert synth.mobilenetv2_pointwise_layers(width=1.0) == base
    assert [synth.scaled_channels(c, 0.75) for c in (16, 24, 32, 64, 96, 160, 320)] == \
        [16, 24, 24, 48, 72, 120, 240]
    assert synth.scaled_channels(24, 1.4) == 32 and synth.scaled_channels(320, 1.4) == 448
    for width in (0.75, 1.25, 1.4, 2.0):
        t = synth.mobilenetv2_pointwise_layers(width=width)
        assert len(t) == len(base)
        for a, b in zip(t, base):
            assert (a.name, a.in_stride, a.h, a.w) == (b.name, b.in_stride, b.h, b.w)
            assert a.cin % 8 == 0 and a.cout % 8 == 0
            if "project" in a.name:
                assert 0.9 * b.cout * width <= a.cout <= b.cout * width + 8
        for prev, cur in zip(t, t[1:]):
            assert cur.cin == prev.cout
        assert t[-1].cout == (1280 if width <= 1.0 else synth.scaled_channels(1280, width))
