"""Pins for the 2-bit weight format: a byte table, round trips, rejection of
invalid values, sizes."""
import numpy as np
import pytest

CODE = {0: 0, 1: 1, -1: 3}
DECODE = {0: 0, 1: 1, 3: -1}


def test_every_byte_value_decodes_by_table(oracle):
    for b in range(256):
        codes = [(b >> (2 * j)) & 3 for j in range(4)]
        w, bad = oracle.unpack(np.array([[b]], np.uint8), 1, 4)
        assert bad == sum(c == 2 for c in codes)
        assert w[0].tolist() == [DECODE.get(c, 0) for c in codes]


def test_pack_layout(oracle):
    # weight k of channel o sits in byte o*ceil(cin/4) + k//4 at bits 2*(k%4)
    w = np.zeros((3, 6), np.int8)
    w[0] = [1, -1, 0, 1, -1, 0]
    w[2, 5] = 1
    p = oracle.pack(w)
    assert p.shape == (3, 2) and p.dtype == np.uint8
    assert p[0].tolist() == [1 | (3 << 2) | (0 << 4) | (1 << 6), 3]
    assert p[1].tolist() == [0, 0]
    assert p[2].tolist() == [0, 1 << 2]


def test_round_trip(oracle):
    rng = np.random.default_rng(0)
    for cout, cin in [(1, 1), (5, 3), (16, 24), (37, 145), (1280, 320)]:
        w = rng.integers(-1, 2, size=(cout, cin), dtype=np.int8)
        p = oracle.pack(w)
        assert p.size == oracle.packed_bytes(cout, cin) == cout * ((cin + 3) // 4)
        w2, bad = oracle.unpack(p, cout, cin)
        assert bad == 0 and np.array_equal(w, w2)
        # python statement of the format
        for o in range(min(cout, 3)):
            for k in range(cin):
                assert (int(p[o, k // 4]) >> (2 * (k % 4))) & 3 == CODE[int(w[o, k])]


def test_invalid_values_rejected(oracle):
    for bad in (2, -2, 127, -128):
        w = np.zeros((2, 8), np.int8)
        w[1, 3] = bad
        with pytest.raises(ValueError):
            oracle.pack(w)


def test_nonzero_padding_is_flagged(oracle):
    p = np.array([[0b01000000]], np.uint8)      # cin = 3: the 4th code must be 00
    _, bad = oracle.unpack(p, 1, 3)
    assert bad == 1


def test_packed_size_of_the_network(oracle):
    from paper_2505_03254_b200 import synth
    total = sum(oracle.packed_bytes(l.cout, l.cin) for l in synth.mobilenetv2_pointwise_layers())
    assert total == 2124672 // 4       # every Cin of the network is a multiple of 4
