"""The layer-sequence oracle against chained single-layer calls with an
explicit gather between them."""
import numpy as np

from paper_2505_03254_b200 import synth


def _mk(seed, shapes):
    layers = []
    for i, (cin, cout, st) in enumerate(shapes):
        d = synth.make_layer(seed, cin, cout, 0.5, index=i + 1)
        layers.append(dict(cin=cin, cout=cout, in_stride=st, w=d["w"].numpy(),
                           bias=d["bias"].numpy(), mult=d["mult"].numpy(),
                           shift=d["shift"].numpy()))
    return layers


def test_subsample_picks_even_pixels(oracle):
    x = np.arange(2 * 4 * 6 * 3, dtype=np.int8).reshape(2, 4, 6, 3)
    assert np.array_equal(oracle.subsample(x, 2), x[:, ::2, ::2, :])
    assert np.array_equal(oracle.subsample(x, 1), x)


def test_sequence_equals_chained_layers(oracle):
    shapes = [(8, 16, 1), (16, 48, 1), (48, 8, 2), (8, 24, 1), (24, 16, 2), (16, 40, 1)]
    layers = _mk(21, shapes)
    x0 = synth.act_post_relu6(21, (3, 8, 12, 8)).numpy()
    got = oracle.layer_seq(layers, x0)
    cur = x0
    for l in layers:
        if l["in_stride"] == 2:
            cur = cur[:, ::2, ::2, :]          # numpy gather, not the oracle's
        b, h, w, c = cur.shape
        y = oracle.conv_mul(np.ascontiguousarray(cur).reshape(-1, c), l["w"], l["bias"],
                            l["mult"], l["shift"])
        cur = y.reshape(b, h, w, l["cout"])
    assert got.shape == (3, 2, 3, 40)
    assert np.array_equal(got, cur)


def test_mobilenetv2_sequence_shapes(oracle):
    table = synth.mobilenetv2_pointwise_layers(h0=16, w0=16)   # same table, small image
    shapes = [(l.cin, l.cout, l.in_stride) for l in table]
    layers = _mk(22, shapes)
    x0 = synth.act_post_relu6(22, (1, 16, 16, 32)).numpy()
    y = oracle.layer_seq(layers, x0)
    assert y.shape == (1, 1, 1, 1280)
    assert y.min() >= 0 and y.max() <= 127
