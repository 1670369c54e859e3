"""ctypes front end of the CPU oracle (``prom_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg import this; the CUDA library and its binding never do.
Arrays are numpy; nothing here computes anything, it only marshals arguments.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "prom_oracle.c")
_LIB = os.path.join(_HERE, "libprom_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``) unless it is up to date."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC",
                           "-Wall", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i8p, u8p, i32p = C.POINTER(C.c_int8), C.POINTER(C.c_uint8), C.POINTER(C.c_int32)
        L.prom_ref_threads.restype = C.c_int
        L.prom_ref_set_threads.argtypes = [C.c_int]
        L.prom_ref_packed_bytes.restype = C.c_size_t
        L.prom_ref_packed_bytes.argtypes = [C.c_int, C.c_int]
        L.prom_ref_pack.restype = C.c_long
        L.prom_ref_pack.argtypes = [i8p, C.c_int, C.c_int, u8p]
        L.prom_ref_unpack.restype = C.c_long
        L.prom_ref_unpack.argtypes = [u8p, C.c_int, C.c_int, i8p]
        L.prom_ref_requant_scalar.restype = C.c_int32
        L.prom_ref_requant_scalar.argtypes = [C.c_int32, C.c_int32, C.c_int, C.c_int, C.c_int]
        L.prom_ref_requant.argtypes = [i32p, C.c_long, C.c_int32, C.c_int, C.c_int, C.c_int, i32p]
        conv = [i8p, C.c_long, C.c_int, C.c_long, i8p, C.c_int, i32p, i32p, i8p,
                C.c_int, C.c_int, i32p, i8p]
        L.prom_ref_conv_mul.argtypes = conv
        L.prom_ref_conv_addsub.argtypes = conv
        L.prom_ref_subsample.argtypes = [i8p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i8p]
        L.prom_ref_residual_add.argtypes = [i8p, i8p, C.c_long, i8p]
        L.prom_ref_layer_seq.restype = C.c_int
        L.prom_ref_layer_seq.argtypes = [
            C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int),
            C.POINTER(i8p), C.POINTER(i32p), C.POINTER(i32p), C.POINTER(i8p),
            C.c_int, C.c_int, i8p, C.c_int, C.c_int, C.c_int, i8p]
        L.prom_ref_quantize_ternary.argtypes = [C.POINTER(C.c_float), C.c_int, C.c_int, C.c_double,
                                                i8p, C.POINTER(C.c_double)]
        L.prom_ref_quantize_act_absmax.argtypes = [C.POINTER(C.c_float), C.c_int, C.c_long, C.c_float,
                                                   i8p, C.POINTER(C.c_float), C.POINTER(C.c_float)]
        L.prom_ref_conv_dyn.argtypes = [i8p, C.c_int, C.c_long, C.c_int, i8p, C.c_int,
                                        C.POINTER(C.c_float), C.POINTER(C.c_float), C.c_float,
                                        C.POINTER(C.c_float), i8p, C.POINTER(C.c_float),
                                        C.POINTER(C.c_float)]
        L.prom_ref_dw3x3.argtypes = [i8p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i8p, i32p, i32p, i8p,
                                     C.c_int, C.c_int, i32p, i8p]
        L.prom_ref_requant_from_scale.restype = C.c_int
        L.prom_ref_requant_from_scale.argtypes = [C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_int)]
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(C.POINTER(ct))


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def threads() -> int:
    return int(lib().prom_ref_threads())


def set_threads(n: int) -> None:
    lib().prom_ref_set_threads(int(n))


def packed_bytes(cout: int, cin: int) -> int:
    return int(lib().prom_ref_packed_bytes(cout, cin))


def pack(w) -> np.ndarray:
    """Ternary int8 [cout, cin] -> 2-bit codes [cout, ceil(cin/4)] (uint8).
    Raises ValueError when an entry is outside {-1, 0, +1}."""
    w = _c(w, np.int8)
    cout, cin = w.shape
    out = np.zeros((cout, (cin + 3) // 4), dtype=np.uint8)
    bad = lib().prom_ref_pack(_p(w, C.c_int8), cout, cin, _p(out, C.c_uint8))
    if bad:
        raise ValueError(f"{bad} weight(s) outside {{-1,0,+1}}")
    return out


def unpack(packed, cout: int, cin: int):
    """2-bit codes -> (ternary int8 [cout, cin], number of invalid codes)."""
    packed = _c(packed, np.uint8).reshape(cout, (cin + 3) // 4)
    w = np.zeros((cout, cin), dtype=np.int8)
    bad = lib().prom_ref_unpack(_p(packed, C.c_uint8), cout, cin, _p(w, C.c_int8))
    return w, int(bad)


def requant_scalar(t: int, mult: int, shift: int, act_min: int = 0, act_max: int = 127) -> int:
    return int(lib().prom_ref_requant_scalar(int(t), int(mult), int(shift), act_min, act_max))


def requant(t, mult: int, shift: int, act_min: int = 0, act_max: int = 127) -> np.ndarray:
    t = _c(t, np.int32).ravel()
    q = np.empty_like(t)
    lib().prom_ref_requant(_p(t, C.c_int32), t.size, int(mult), int(shift), act_min, act_max,
                           _p(q, C.c_int32))
    return q


def _conv(fn, x, w, bias, mult, shift, act_min, act_max, want_acc, want_y):
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    m, cin = x.shape
    cout, cin2 = w.shape
    assert cin == cin2
    bias = _c(bias, np.int32)
    mult = _c(mult, np.int32)
    shift = _c(shift, np.int8)
    assert bias.size == cout and mult.size == cout and shift.size == cout
    acc = np.empty((m, cout), dtype=np.int32) if want_acc else None
    y = np.empty((m, cout), dtype=np.int8) if want_y else None
    fn(_p(x, C.c_int8), m, cin, cin, _p(w, C.c_int8), cout,
       _p(bias, C.c_int32), _p(mult, C.c_int32), _p(shift, C.c_int8),
       act_min, act_max,
       _p(acc, C.c_int32) if want_acc else None,
       _p(y, C.c_int8) if want_y else None)
    return acc, y


def conv_mul(x, w, bias, mult, shift, act_min=0, act_max=127, want_acc=False):
    """Multiply form. Returns y [m, cout] int8 (and acc int32 when want_acc)."""
    acc, y = _conv(lib().prom_ref_conv_mul, x, w, bias, mult, shift, act_min, act_max,
                   want_acc, True)
    return (y, acc) if want_acc else y


def conv_addsub(x, w, bias, mult, shift, act_min=0, act_max=127, want_acc=False):
    """Add/subtract form of the same layer."""
    acc, y = _conv(lib().prom_ref_conv_addsub, x, w, bias, mult, shift, act_min, act_max,
                   want_acc, True)
    return (y, acc) if want_acc else y


def subsample(x, stride: int) -> np.ndarray:
    x = _c(x, np.int8)
    b, h, w, c = x.shape
    out = np.empty((b, h // stride, w // stride, c), dtype=np.int8)
    lib().prom_ref_subsample(_p(x, C.c_int8), b, h, w, c, stride, _p(out, C.c_int8))
    return out


def residual_add(y_layer, block_in) -> np.ndarray:
    """Skip connection (Section 2): clamp(y_layer + block_in, -128, 127), int8 arrays of one shape."""
    a, b = _c(y_layer, np.int8), _c(block_in, np.int8)
    assert a.shape == b.shape
    out = np.empty_like(a)
    lib().prom_ref_residual_add(_p(a, C.c_int8), _p(b, C.c_int8), a.size, _p(out, C.c_int8))
    return out


def layer_seq(layers, x0, act_min=0, act_max=127) -> np.ndarray:
    """layers: list of dicts with cin, cout, in_stride, w (ternary int8 [cout, cin]),
    bias, mult, shift.  x0: [batch, h0, w0, cin0] int8.  Returns the last
    layer's output [batch, h, w, cout]."""
    x0 = _c(x0, np.int8)
    batch, h0, w0, c0 = x0.shape
    n = len(layers)
    assert c0 == layers[0]["cin"]
    ws = [_c(l["w"], np.int8) for l in layers]
    bs = [_c(l["bias"], np.int32) for l in layers]
    ms = [_c(l["mult"], np.int32) for l in layers]
    ss = [_c(l["shift"], np.int8) for l in layers]
    IA = C.c_int * n
    cin = IA(*[int(l["cin"]) for l in layers])
    cout = IA(*[int(l["cout"]) for l in layers])
    st = IA(*[int(l["in_stride"]) for l in layers])
    i8p, i32p = C.POINTER(C.c_int8), C.POINTER(C.c_int32)
    wp = (i8p * n)(*[_p(a, C.c_int8) for a in ws])
    bp = (i32p * n)(*[_p(a, C.c_int32) for a in bs])
    mp = (i32p * n)(*[_p(a, C.c_int32) for a in ms])
    sp = (i8p * n)(*[_p(a, C.c_int8) for a in ss])
    h, w = h0, w0
    for l in layers:
        h //= l["in_stride"]
        w //= l["in_stride"]
    y = np.empty((batch, h, w, layers[-1]["cout"]), dtype=np.int8)
    rc = lib().prom_ref_layer_seq(n, cin, cout, st, wp, bp, mp, sp, act_min, act_max,
                                  _p(x0, C.c_int8), batch, h0, w0, _p(y, C.c_int8))
    if rc != 0:
        raise ValueError("layer sequence does not chain")
    return y


def quantize_ternary(w, eps: float = 1e-5):
    """Absmean ternary quantiser (paper Eq. 1-3 / Figure 10).  w: float32 [cout, cin].
    Returns (q int8 [cout, cin] in {-1,0,+1}, alpha float64 [cout])."""
    w = _c(w, np.float32)
    cout, cin = w.shape
    q = np.empty((cout, cin), dtype=np.int8)
    alpha = np.empty((cout,), dtype=np.float64)
    lib().prom_ref_quantize_ternary(_p(w, C.c_float), cout, cin, float(eps), _p(q, C.c_int8),
                                    _p(alpha, C.c_double))
    return q, alpha


def requant_from_scale(scale: float):
    """(mult, shift) with mult in [2^30, 2^31) and mult * 2^-(31+shift) nearest to scale."""
    m, s = C.c_int32(), C.c_int()
    if lib().prom_ref_requant_from_scale(float(scale), C.byref(m), C.byref(s)) != 0:
        raise ValueError("scale cannot be represented with a shift in [0, 31]")
    return int(m.value), int(s.value)


def quantize_act_absmax(x, eps: float = 1e-5):
    """Per-sample absmax quantiser of activations (paper Eq. 6-7 / the activation figure of
    the pseudocode appendix).  x: float32 [batch, ...].  Returns (q int8 like x,
    gamma float32 [batch] = max |x| per sample, scale float32 [batch] = 127 / max(gamma, eps))."""
    x = _c(x, np.float32)
    batch = x.shape[0]
    per = int(np.prod(x.shape[1:])) if x.ndim > 1 else 1
    q = np.empty(x.shape, dtype=np.int8)
    gamma = np.empty((batch,), dtype=np.float32)
    scale = np.empty((batch,), dtype=np.float32)
    lib().prom_ref_quantize_act_absmax(_p(x, C.c_float), batch, C.c_long(per), C.c_float(eps),
                                       _p(q, C.c_int8), _p(gamma, C.c_float), _p(scale, C.c_float))
    return q, gamma, scale


def conv_dyn(x, w, alpha, gamma_x, rows_per_sample: int, eps: float = 1e-5):
    """A pointwise layer in the paper's inference dataflow: ternary convolution of quantised
    activations, dequantised by alpha[o] and the input's per-sample scale, then quantised again
    per sample.  x: int8 [batch * rows_per_sample, cin]; w: int8 [cout, cin] ternary; alpha:
    float32 [cout]; gamma_x: float32 [batch].  Returns (q int8 [m, cout], gamma_y, scale_y
    float32 [batch], y float32 [m, cout])."""
    x = _c(x, np.int8); w = _c(w, np.int8)
    alpha = _c(alpha, np.float32); gamma_x = _c(gamma_x, np.float32)
    m, cin = x.shape
    cout = w.shape[0]
    batch = gamma_x.shape[0]
    assert m == batch * rows_per_sample and w.shape[1] == cin and alpha.shape[0] == cout
    y = np.empty((m, cout), dtype=np.float32)
    q = np.empty((m, cout), dtype=np.int8)
    gy = np.empty((batch,), dtype=np.float32)
    sy = np.empty((batch,), dtype=np.float32)
    lib().prom_ref_conv_dyn(_p(x, C.c_int8), batch, C.c_long(rows_per_sample), cin, _p(w, C.c_int8), cout,
                            _p(alpha, C.c_float), _p(gamma_x, C.c_float), C.c_float(eps),
                            _p(y, C.c_float), _p(q, C.c_int8), _p(gy, C.c_float), _p(sy, C.c_float))
    return q, gy, sy, y


def dw3x3(x, w, bias, mult, shift, stride: int = 1, act_min: int = -128, act_max: int = 127,
          want_acc: bool = False):
    """int8 depthwise 3x3 convolution, zero padding 1, per-channel fixed-point requantisation.
    x: int8 [batch, h, w, c]; w: int8 [c, 3, 3]; bias, mult int32 [c]; shift int8 [c].
    Returns y int8 [batch, ho, wo, c] (and the int32 accumulators when want_acc)."""
    x = _c(x, np.int8); w = _c(w, np.int8)
    bias = _c(bias, np.int32); mult = _c(mult, np.int32); shift = _c(shift, np.int8)
    b, h, wd, c = x.shape
    assert w.shape == (c, 3, 3) and stride in (1, 2)
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    y = np.empty((b, ho, wo, c), dtype=np.int8)
    acc = np.empty((b, ho, wo, c), dtype=np.int32) if want_acc else None
    lib().prom_ref_dw3x3(_p(x, C.c_int8), b, h, wd, c, stride, _p(w, C.c_int8), _p(bias, C.c_int32),
                         _p(mult, C.c_int32), _p(shift, C.c_int8), act_min, act_max,
                         _p(acc, C.c_int32) if want_acc else None, _p(y, C.c_int8))
    return (y, acc) if want_acc else y
