"""Seeded synthetic inputs for the ternary pointwise-convolution path.

This module holds no arithmetic of the method itself: it only draws the
tensors the path consumes (activations, ternary weights, requantisation
constants) and lists the layer shapes of the workloads.  Both the CUDA path's
tests/benchmark and the CPU oracle's tests take their inputs from here.

Every stream is a counter-based hash, so any element can be regenerated on
its own, on the host or on the device:

    h(seed, stream, i) = mix(seed + GOLDEN*(i+1) + STREAM_MUL*stream)  (mod 2^64)

with ``mix`` the SplitMix64 output function (Steele, Lea, Flood 2014) and
``i`` the flat element index.  The tensors stand in for ImageNet-trained
MobileNetV2 layers: they take the layer shapes of MobileNetV2-1.0 at 224x224,
the value range of int8 activations after a ReLU6 (uniform on [0,127] with
30 % exact zeros) and the ternary statistics the paper reports (about a third
zeros at initialisation, up to 55 % after training, +1 and -1 balanced).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import torch

GOLDEN = 0x9E3779B97F4A7C15
STREAM_MUL = 0xD1B54A32D192ED03
MIX1 = 0xBF58476D1CE4E5B9
MIX2 = 0x94D049BB133111EB
BASE_SEED = 0x50524F4D  # "PROM"

STREAM_X, STREAM_W, STREAM_BIAS, STREAM_MULT, STREAM_SHIFT = 1, 2, 3, 4, 5

_MASK64 = (1 << 64) - 1
_CHUNK = 1 << 24


def _s64(v: int) -> int:
    """Two's-complement view of a 64-bit pattern as a Python int torch accepts."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (z >> n) & ((1 << (64 - n)) - 1)


def hash64(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """h(seed, stream, i) for i in [start, start+count) as int64 bit patterns."""
    i = torch.arange(start + 1, start + count + 1, dtype=torch.int64, device=device)
    z = i * _s64(GOLDEN) + _s64(seed + STREAM_MUL * stream)
    z = (z ^ _lsr(z, 30)) * _s64(MIX1)
    z = (z ^ _lsr(z, 27)) * _s64(MIX2)
    return z ^ _lsr(z, 31)


def _fill(n: int, device, dtype, fn) -> torch.Tensor:
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        out[s:s + c] = fn(s, c)
    return out


def _threshold(frac: float) -> int:
    return int(frac * 4294967296.0)  # floor(frac * 2^32)


def act_uniform_i8(seed: int, shape, device="cpu", stream: int = STREAM_X) -> torch.Tensor:
    """int8 activations uniform on [-128, 127]."""
    n = 1
    for d in shape:
        n *= int(d)

    def fn(s, c):
        h = hash64(seed, stream, s, c, device)
        return ((h & 0xFF) ^ 0x80) - 0x80  # low byte reinterpreted as signed

    return _fill(n, device, torch.int8, fn).view(*shape)


def act_uniform_0_127(seed: int, shape, device="cpu", stream: int = STREAM_X) -> torch.Tensor:
    """int8 activations uniform on [0, 127]."""
    n = 1
    for d in shape:
        n *= int(d)
    return _fill(n, device, torch.int8,
                 lambda s, c: hash64(seed, stream, s, c, device) & 0x7F).view(*shape)


def act_post_relu6(seed: int, shape, device="cpu", zero_frac: float = 0.3,
                   stream: int = STREAM_X) -> torch.Tensor:
    """Post-ReLU6 distribution: uniform on [0,127], then an independent
    ``zero_frac`` of the entries forced to 0."""
    n = 1
    for d in shape:
        n *= int(d)
    thr = _threshold(zero_frac)

    def fn(s, c):
        h = hash64(seed, stream, s, c, device)
        v = h & 0x7F
        return torch.where(_lsr(h, 32) < thr, torch.zeros_like(v), v)

    return _fill(n, device, torch.int8, fn).view(*shape)


def ternary_weights(seed: int, cout: int, cin: int, zero_frac: float = 0.5, device="cpu",
                    stream: int = STREAM_W) -> torch.Tensor:
    """iid ternary [cout, cin] int8: P(0)=zero_frac, P(+1)=P(-1)=(1-zero_frac)/2."""
    thr = _threshold(zero_frac)

    def fn(s, c):
        h = hash64(seed, stream, s, c, device)
        pm = (h & 1) * 2 - 1
        return torch.where(_lsr(h, 32) < thr, torch.zeros_like(pm), pm)

    return _fill(cout * cin, device, torch.int8, fn).view(cout, cin)


def requant_constants(seed: int, cout: int, device="cpu", stream_base: int = 0):
    """(bias int32 uniform on [-4096, 4096], mult int32 uniform on [2^30, 2^31),
    shift int8 uniform on {8..12}), each [cout]."""
    hb = hash64(seed, stream_base + STREAM_BIAS, 0, cout, device)
    hm = hash64(seed, stream_base + STREAM_MULT, 0, cout, device)
    hs = hash64(seed, stream_base + STREAM_SHIFT, 0, cout, device)
    bias = (_lsr(hb, 11) % 8193 - 4096).to(torch.int32)
    mult = ((1 << 30) + (hm & ((1 << 30) - 1))).to(torch.int32)
    shift = (8 + _lsr(hs, 40) % 5).to(torch.int8)
    return bias, mult, shift


# ---------------------------------------------------------------------------
# workloads
# ---------------------------------------------------------------------------

@dataclass(frozen=True)
class LayerShape:
    name: str
    cin: int
    cout: int
    in_stride: int   # spatial subsample applied to this layer's input (1 or 2)
    h: int           # spatial size this layer runs at (after in_stride)
    w: int


MOBILENETV2_TCNS = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                    (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]


def scaled_channels(channels: int, width: float, divisor: int = 8) -> int:
    """Channel count under a width multiplier: the nearest multiple of `divisor`
    (at least `divisor`), raised by one step where rounding would lose more than a
    tenth of the scaled count.  This is the usual rule of MobileNet-family models."""
    v = channels * width
    c = max(divisor, int(v + divisor / 2) // divisor * divisor)
    if c < 0.9 * v:
        c += divisor
    return c


def mobilenetv2_pointwise_layers(stem_channels: int = 32, h0: int = 112, w0: int = 112,
                                 head_channels: int = 1280, width: float = 1.0) -> List[LayerShape]:
    """Every 1x1 convolution of MobileNetV2: per inverted-residual block a ternary
    expand (omitted when t = 1) and a ternary project, then the head convolution.
    The block's stride sits in its depthwise convolution, so the project after a
    stride-2 depthwise reads a subsampled input.  `width` scales every channel count
    (Section 5, Experiments: widths 0.75x to 2.0x); the head only grows, for widths above one."""
    layers: List[LayerShape] = []
    c, h, w = stem_channels, h0, w0
    if width != 1.0:
        c = scaled_channels(stem_channels, width)
        head_channels = scaled_channels(head_channels, max(1.0, width))
    for bi, (t, cout, n, s) in enumerate(MOBILENETV2_TCNS, start=1):
        if width != 1.0:
            cout = scaled_channels(cout, width)
        for r in range(n):
            stride = s if r == 0 else 1
            hidden = c * t
            if t != 1:
                layers.append(LayerShape(f"b{bi}.{r + 1}.expand", c, hidden, 1, h, w))
            h, w = h // stride, w // stride
            layers.append(LayerShape(f"b{bi}.{r + 1}.project", hidden, cout, stride, h, w))
            c = cout
    layers.append(LayerShape("head", c, head_channels, 1, h, w))
    return layers


def has_skip_connection(layers: List[LayerShape], i: int) -> bool:
    """Whether layer i of `mobilenetv2_pointwise_layers` closes a block that keeps its input's
    shape (stride 1, equal channel counts): the block's input is then added to its output."""
    return (i > 0 and layers[i].name.endswith("project") and layers[i - 1].name.endswith("expand")
            and layers[i].in_stride == 1 and layers[i - 1].in_stride == 1
            and layers[i].cout == layers[i - 1].cin)


def layer_seed(seed: int, index: int) -> int:
    """Seed offset of layer `index` in a sequence (streams 1000*index + s)."""
    return 1000 * index


def make_layer(seed: int, cin: int, cout: int, zero_frac: float = 0.5, device="cpu",
               index: int = 0):
    """Ternary weights and requantisation constants of one layer."""
    base = layer_seed(seed, index)
    w = ternary_weights(seed, cout, cin, zero_frac, device, stream=base + STREAM_W)
    bias, mult, shift = requant_constants(seed, cout, device, stream_base=base)
    return dict(cin=cin, cout=cout, w=w, bias=bias, mult=mult, shift=shift)


CONFIG5_CIN = (16, 64, 144, 384, 960)
CONFIG5_COUT = (24, 96, 320, 1280)
CONFIG5_M = (12544, 200704, 1605632)
CONFIG5_ZERO = (0.3, 0.5, 0.7, 0.9)
CONFIG4_SHAPES = ((960, 160), (160, 960), (320, 1280))
