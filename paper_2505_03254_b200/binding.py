"""Thin ctypes binding over the C-ABI library (``include/prom.h``).

Argument marshalling only: every function hands device (or host) pointers of
torch tensors to the entry point of the same name; all arithmetic runs in the
library's CUDA kernels.  There is no fallback: if the library is missing, or a
tensor lives on the wrong device, the call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprom.so")

PROM_OK = 0
(PROM_ERR_NULL, PROM_ERR_SHAPE, PROM_ERR_ALIGN, PROM_ERR_BAD_WEIGHT, PROM_ERR_BAD_REQUANT,
 PROM_ERR_WORKSPACE, PROM_ERR_UNSUPPORTED, PROM_ERR_CUDA, PROM_ERR_TIMEOUT) = range(1, 10)

VARIANTS = {"auto": 0, "tc": 1, "smallk": 2, "addsub": 3, "naive": 4}

EXPORTS = [
    "prom_packed_bytes", "prom_pack_ternary", "prom_pw_conv_i8", "prom_pw_conv_i8_acc32",
    "prom_pw_conv_i8_host", "prom_layer_seq_workspace_bytes", "prom_pw_layer_seq",
    "prom_layer_seq_host_workspace_bytes", "prom_pw_layer_seq_host", "prom_last_device_status",
    "prom_launch_count", "prom_shutdown", "prom_status_string",
    "prom_pw_conv_i8_addsub_static", "prom_debug_tc_plan", "prom_debug_tc_plan_query",
    "prom_quantize_ternary", "prom_requant_from_scale", "prom_quantize_act_absmax", "prom_pw_conv_i8_dyn", "prom_dw_conv3x3_i8", "prom_debug_tc_plan_shape", "prom_pw_conv_i8_res",
    "prom_debug_seq_chain", "prom_debug_seq_order", "prom_debug_wait_timeout", "prom_debug_i8_mma_rate", "prom_debug_alu_rate",
    "prom_debug_once_per_device", "prom_debug_layer_seq_output_offset",
    "prom_pw_prepared_bytes", "prom_pw_prepare", "prom_pw_conv_i8_prepared", "prom_quantize_ternary_batch",
    "prom_debug_dw_variant", "prom_debug_tc_wide", "prom_debug_mma_issue_rate", "prom_debug_l2_copy_rate",
    "prom_debug_mma_beside",
]
STATIC_SCRATCH_BYTES = 6 << 20


class PromRequant(C.Structure):
    _fields_ = [("bias", C.c_void_p), ("mult", C.c_void_p), ("shift", C.c_void_p),
                ("act_min", C.c_int), ("act_max", C.c_int)]


class PromLayer(C.Structure):
    _fields_ = [("cin", C.c_int), ("cout", C.c_int), ("in_stride", C.c_int),
                ("w_packed", C.c_void_p), ("rq", PromRequant),
                ("dw_w", C.c_void_p), ("dw_rq", PromRequant), ("add_block_input", C.c_int)]


class PromQuantizeJob(C.Structure):
    _fields_ = [("w_dev", C.c_void_p), ("cout", C.c_int), ("cin", C.c_int), ("packed_dev", C.c_void_p),
                ("packed_bytes", C.c_size_t), ("alpha_dev", C.c_void_p)]


class PromError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} (prom_status {code})")
        self.code = code


_lib = None


def lib():
    """Loads ``libprom.so`` (built in-tree by ``build.build()``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run paper_2505_03254_b200.build.build()")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
        L.prom_packed_bytes.restype = sz
        L.prom_packed_bytes.argtypes = [i32, i32]
        L.prom_pack_ternary.restype = i32
        L.prom_pack_ternary.argtypes = [vp, i32, i32, vp, sz, vp]
        L.prom_pw_conv_i8.restype = i32
        L.prom_pw_conv_i8.argtypes = [vp, i64, i32, vp, i32, C.POINTER(PromRequant), vp, i32, vp]
        L.prom_pw_prepared_bytes.restype = sz
        L.prom_pw_prepared_bytes.argtypes = [i64, i32, i32]
        L.prom_pw_prepare.restype = i32
        L.prom_pw_prepare.argtypes = [i64, i32, vp, i32, C.POINTER(PromRequant), vp, sz, vp]
        L.prom_pw_conv_i8_prepared.restype = i32
        L.prom_pw_conv_i8_prepared.argtypes = [vp, i64, i32, i32, vp, i32, i32, vp, vp]
        L.prom_pw_conv_i8_res.restype = i32
        L.prom_pw_conv_i8_res.argtypes = [vp, i64, i32, vp, i32, C.POINTER(PromRequant), vp, vp, i32, vp]
        L.prom_pw_conv_i8_acc32.restype = i32
        L.prom_pw_conv_i8_acc32.argtypes = [vp, i64, i32, vp, i32, vp, vp]
        L.prom_pw_conv_i8_host.restype = i32
        L.prom_pw_conv_i8_host.argtypes = [vp, i64, i32, vp, i32, C.POINTER(PromRequant), vp,
                                           vp, sz, i32, vp]
        L.prom_layer_seq_workspace_bytes.restype = sz
        L.prom_layer_seq_workspace_bytes.argtypes = [C.POINTER(PromLayer), i32, i32, i32, i32]
        L.prom_pw_layer_seq.restype = i32
        L.prom_pw_layer_seq.argtypes = [C.POINTER(PromLayer), i32, vp, i32, i32, i32, vp, sz, vp,
                                        i32, vp]
        L.prom_layer_seq_host_workspace_bytes.restype = sz
        L.prom_layer_seq_host_workspace_bytes.argtypes = [C.POINTER(PromLayer), i32, i32, i32, i32]
        L.prom_pw_layer_seq_host.restype = i32
        L.prom_pw_layer_seq_host.argtypes = [C.POINTER(PromLayer), i32, vp, i32, i32, i32, vp, sz,
                                             vp, i32, vp]
        L.prom_pw_conv_i8_addsub_static.restype = i32
        L.prom_pw_conv_i8_addsub_static.argtypes = [vp, i64, i32, vp, i32, C.POINTER(PromRequant),
                                                    vp, vp]
        L.prom_dw_conv3x3_i8.restype = i32
        L.prom_dw_conv3x3_i8.argtypes = [C.c_void_p, i32, i32, i32, i32, i32, C.c_void_p, C.POINTER(PromRequant),
                                         C.c_void_p, C.c_void_p]
        L.prom_pw_conv_i8_dyn.restype = i32
        L.prom_pw_conv_i8_dyn.argtypes = [C.c_void_p, i32, i64, i32, C.c_void_p, i32, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.prom_quantize_act_absmax.restype = i32
        L.prom_quantize_act_absmax.argtypes = [C.c_void_p, i32, i64, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p]
        L.prom_debug_tc_plan_shape.restype = None
        L.prom_debug_tc_plan_shape.argtypes = [i64, i32, i32, i32, i32, i32, i32, i32, i32]
        L.prom_debug_tc_plan.restype = None
        L.prom_debug_tc_plan.argtypes = [i32, i32, i32, i32, i32]
        L.prom_debug_tc_plan_query.restype = i32
        L.prom_debug_tc_plan_query.argtypes = [i64, i32, i32, C.POINTER(C.c_int)]
        L.prom_debug_dw_variant.restype = None
        L.prom_debug_dw_variant.argtypes = [i32]
        L.prom_debug_tc_wide.restype = None
        L.prom_debug_tc_wide.argtypes = [i32, i32]
        L.prom_debug_seq_chain.restype = None
        L.prom_debug_seq_chain.argtypes = [i32]
        L.prom_debug_seq_order.restype = None
        L.prom_debug_seq_order.argtypes = [i32]
        L.prom_debug_layer_seq_output_offset.restype = i64
        L.prom_debug_layer_seq_output_offset.argtypes = [C.POINTER(PromLayer), i32, i32, i32, i32, i32,
                                                         C.POINTER(C.c_int)]
        L.prom_debug_wait_timeout.restype = i32
        L.prom_debug_wait_timeout.argtypes = [C.c_uint64, vp, vp]
        L.prom_debug_i8_mma_rate.restype = i32
        L.prom_debug_i8_mma_rate.argtypes = [i32, vp, i32, C.POINTER(C.c_int), vp]
        L.prom_debug_alu_rate.restype = i32
        L.prom_debug_alu_rate.argtypes = [i32, i32, vp, vp, i32, C.POINTER(C.c_int), vp]
        L.prom_debug_mma_issue_rate.restype = i32
        L.prom_debug_mma_issue_rate.argtypes = [i32, i32, i32, vp, i32, C.POINTER(C.c_int), vp]
        L.prom_debug_l2_copy_rate.restype = i32
        L.prom_debug_l2_copy_rate.argtypes = [vp, C.c_uint64, i32, i32, vp, i32, C.POINTER(C.c_int), vp]
        L.prom_debug_mma_beside.restype = i32
        L.prom_debug_mma_beside.argtypes = [i32, i32, i32, i32, vp, C.c_uint64, vp, i32, C.POINTER(C.c_int), vp]
        L.prom_debug_once_per_device.restype = i32
        L.prom_debug_once_per_device.argtypes = [i32, i32]
        L.prom_quantize_ternary_batch.restype = i32
        L.prom_quantize_ternary_batch.argtypes = [C.POINTER(PromQuantizeJob), i32, vp]
        L.prom_quantize_ternary.restype = i32
        L.prom_quantize_ternary.argtypes = [vp, i32, i32, vp, sz, vp, vp]
        L.prom_requant_from_scale.restype = i32
        L.prom_requant_from_scale.argtypes = [C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_int8)]
        L.prom_last_device_status.restype = i32
        L.prom_last_device_status.argtypes = [vp]
        L.prom_launch_count.restype = C.c_uint64
        L.prom_shutdown.restype = None
        L.prom_status_string.restype = C.c_char_p
        L.prom_status_string.argtypes = [i32]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().prom_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != PROM_OK:
        raise PromError(code, what)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous {dtype}")
    return t.data_ptr()


def _variant(v) -> int:
    return VARIANTS[v] if isinstance(v, str) else int(v)


def packed_bytes(cout: int, cin: int) -> int:
    return int(lib().prom_packed_bytes(cout, cin))


def launch_count() -> int:
    return int(lib().prom_launch_count())


def last_device_status(stream=None) -> int:
    return int(lib().prom_last_device_status(_stream(stream)))


def dw_conv3x3_i8(x: torch.Tensor, w: torch.Tensor, rq: "PromRequant", stride: int = 1, y=None, stream=None):
    """prom_dw_conv3x3_i8: x int8 [batch, h, w, c], w int8 [c, 3, 3] on the device ->
    y int8 [batch, ho, wo, c]."""
    b, h, wd, c = x.shape
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    if y is None:
        y = torch.empty((b, ho, wo, c), dtype=torch.int8, device=x.device)
    _check(lib().prom_dw_conv3x3_i8(_dev(x, torch.int8, "x"), b, h, wd, c, stride, _dev(w, torch.int8, "w"),
                                    C.byref(rq), _dev(y, torch.int8, "y"), _stream(stream)),
           "prom_dw_conv3x3_i8")
    return y


def pw_conv_i8_dyn(x: torch.Tensor, batch: int, w_packed: torch.Tensor, cout: int, alpha: torch.Tensor,
                   gamma_x: torch.Tensor, out=None, stream=None):
    """prom_pw_conv_i8_dyn: x int8 [batch * rows_per_sample, cin], alpha float32 [cout], gamma_x
    float32 [batch], all on the device -> (q int8 [m, cout], gamma_y, scale_y float32 [batch])."""
    m, cin = x.shape
    if batch and m % batch:
        raise ValueError("rows must divide evenly into samples")
    rows = m // batch if batch else 1
    if out is None:
        q = torch.empty((m, cout), dtype=torch.int8, device=x.device)
        gy = torch.empty((batch,), dtype=torch.float32, device=x.device)
        sy = torch.empty((batch,), dtype=torch.float32, device=x.device)
    else:
        q, gy, sy = out
    _check(lib().prom_pw_conv_i8_dyn(_dev(x, torch.int8, "x"), batch, rows, cin,
                                     _dev(w_packed, torch.uint8, "w_packed"), cout,
                                     _dev(alpha, torch.float32, "alpha"), _dev(gamma_x, torch.float32, "gamma_x"),
                                     q.data_ptr(), gy.data_ptr(), sy.data_ptr(), _stream(stream)),
           "prom_pw_conv_i8_dyn")
    return q, gy, sy


def quantize_act_absmax(x: torch.Tensor, out=None, stream=None):
    """prom_quantize_act_absmax: float32 activations [batch, ...] on the device -> (q int8 like
    x, gamma float32 [batch], scale float32 [batch]); `out` may carry the three tensors."""
    if not x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous():
        raise ValueError("x must be a contiguous float32 CUDA tensor")
    batch = x.shape[0]
    per = x.numel() // batch if batch else 1
    if out is None:
        q = torch.empty(x.shape, dtype=torch.int8, device=x.device)
        gamma = torch.empty((batch,), dtype=torch.float32, device=x.device)
        scale = torch.empty((batch,), dtype=torch.float32, device=x.device)
    else:
        q, gamma, scale = out
        if q.shape != x.shape or q.dtype != torch.int8 or not q.is_cuda or gamma.numel() != batch or \
                scale.numel() != batch or gamma.dtype != torch.float32 or scale.dtype != torch.float32:
            raise ValueError("out must be (int8 like x, float32 [batch], float32 [batch]) on the device")
    _check(lib().prom_quantize_act_absmax(x.data_ptr(), batch, per, q.data_ptr(), gamma.data_ptr(),
                                          scale.data_ptr(), _stream(stream)), "prom_quantize_act_absmax")
    return q, gamma, scale


def debug_tc_plan(fold: int = 0, nt: int = 0, groups: int = 0, occ: int = 0, stages: int = 0) -> None:
    """prom_debug_tc_plan: force parts of the tensor-core launch plan (0 = automatic)."""
    lib().prom_debug_tc_plan(fold, nt, groups, occ, stages)


def debug_tc_plan_shape(m: int, cin: int, cout: int, stride: int = 1, fold: int = 0, nt: int = 0,
                        groups: int = 0, occ: int = 0, stages: int = 0) -> None:
    """prom_debug_tc_plan_shape: force parts of the plan of one shape (all 0 removes the override)."""
    lib().prom_debug_tc_plan_shape(m, cin, cout, stride, fold, nt, groups, occ, stages)


def debug_tc_plan_query(m: int, cin: int, cout: int):
    """prom_debug_tc_plan_query: the plan for a plain layer as a dict, or None."""
    out = (C.c_int * 9)()
    if not lib().prom_debug_tc_plan_query(m, cin, cout, out):
        return None
    keys = ("fold", "nt", "groups", "grid", "stages", "nbuf", "smem", "cw", "est_us_x100")
    return dict(zip(keys, list(out)))


def debug_dw_variant(variant: int = 0) -> None:
    """prom_debug_dw_variant: 0 = the library's choice, 1 = CUDA cores, 2 = tensor cores or refuse."""
    lib().prom_debug_dw_variant(int(variant))


def debug_tc_wide(mode: int = 0, blocks: int = 0) -> None:
    """prom_debug_tc_wide: mode 0 = the library's choice, 1 = the weight-resident kernel only, 2 = the
    row-resident kernel or refuse; blocks = 128-channel blocks per column tile of that kernel (1, 2,
    0 = the planner's choice)."""
    lib().prom_debug_tc_wide(int(mode), int(blocks))


def debug_seq_chain(mode: int = 0) -> None:
    """prom_debug_seq_chain: 0 = one launch per layer (default), 1 = depth-first launches for
    every run of layers that qualifies, 2 = runs whose activations stay in shared memory."""
    lib().prom_debug_seq_chain(int(mode))


def debug_seq_order(alternate: bool = True) -> None:
    """prom_debug_seq_order: whether every second layer of a sequence walks its row tiles backwards
    (the default)."""
    lib().prom_debug_seq_order(1 if alternate else 0)


def debug_layer_seq_output_offset(seq: "LayerSeq", batch: int, h0: int, w0: int, layer: int):
    """prom_debug_layer_seq_output_offset: (byte offset of the layer's output in the workspace, -1
    for a bad argument or -2 for a layer inside a shared-memory run, which writes no tensor;
    whether the layer runs inside a multi-layer launch)."""
    chained = C.c_int(0)
    off = lib().prom_debug_layer_seq_output_offset(seq.array, seq.n, batch, h0, w0, layer, C.byref(chained))
    return int(off), bool(chained.value)


def debug_wait_timeout(limit_ns: int = 5000, stream=None) -> int:
    """prom_debug_wait_timeout: a bounded wait that is left to run out; returns 1 when the
    wait gave up (read back after a synchronise)."""
    flag = torch.zeros((1,), dtype=torch.int32, device="cuda")
    _check(lib().prom_debug_wait_timeout(int(limit_ns), flag.data_ptr(), _stream(stream)),
           "prom_debug_wait_timeout")
    torch.cuda.synchronize()
    return int(flag.item())


def debug_i8_mma_rate(iters: int, cycles: torch.Tensor, stream=None) -> int:
    """prom_debug_i8_mma_rate: launches the tensor-pipe probe; cycles is an int64 CUDA tensor
    that receives per-CTA SM clocks.  Returns the grid size."""
    grid = C.c_int(0)
    _check(lib().prom_debug_i8_mma_rate(int(iters), _dev(cycles, torch.int64, "cycles"), cycles.numel(),
                                        C.byref(grid), _stream(stream)), "prom_debug_i8_mma_rate")
    return int(grid.value)


def debug_alu_rate(op: int, iters: int, sink: torch.Tensor, cycles: torch.Tensor, stream=None) -> int:
    """prom_debug_alu_rate: op 0 mul.hi.s32, 1 mad.lo.s32, 2 fma.rn.f32.  Returns the grid size."""
    grid = C.c_int(0)
    _check(lib().prom_debug_alu_rate(int(op), int(iters), _dev(sink, torch.int32, "sink"),
                                     _dev(cycles, torch.int64, "cycles"), cycles.numel(), C.byref(grid),
                                     _stream(stream)), "prom_debug_alu_rate")
    return int(grid.value)


def debug_mma_issue_rate(n: int, warps: int, iters: int, cycles: torch.Tensor, stream=None) -> int:
    """prom_debug_mma_issue_rate: cycles[4 * cta + w] = SM clocks of issuing warp w.  Returns the grid size."""
    grid = C.c_int(0)
    _check(lib().prom_debug_mma_issue_rate(int(n), int(warps), int(iters), _dev(cycles, torch.int64, "cycles"),
                                           cycles.numel(), C.byref(grid), _stream(stream)),
           "prom_debug_mma_issue_rate")
    return int(grid.value)


def debug_l2_copy_rate(region: torch.Tensor, iters: int, stages: int, cycles: torch.Tensor, stream=None) -> int:
    """prom_debug_l2_copy_rate: every SM copies 16 KB pieces of `region` (device uint8) into its shared
    memory, `stages` at a time.  Returns the grid size."""
    grid = C.c_int(0)
    _check(lib().prom_debug_l2_copy_rate(_dev(region, torch.uint8, "region"), region.numel(), int(iters),
                                         int(stages), _dev(cycles, torch.int64, "cycles"), cycles.numel(),
                                         C.byref(grid), _stream(stream)), "prom_debug_l2_copy_rate")
    return int(grid.value)


def debug_mma_beside(mode: int, iters: int, nwarps: int, stages: int, region, out: torch.Tensor, stream=None) -> int:
    """prom_debug_mma_beside: MMAs beside bulk copies (mode 0) or beside tensor-memory reads (mode 1);
    out[8 * cta + i] as in the header.  Returns the grid size."""
    grid = C.c_int(0)
    rp = _dev(region, torch.uint8, "region") if region is not None else None
    rb = region.numel() if region is not None else 0
    _check(lib().prom_debug_mma_beside(int(mode), int(iters), int(nwarps), int(stages), rp, rb,
                                       _dev(out, torch.int64, "out"), out.numel(), C.byref(grid), _stream(stream)),
           "prom_debug_mma_beside")
    return int(grid.value)


def debug_once_per_device(device: int, key: int) -> bool:
    return bool(lib().prom_debug_once_per_device(int(device), int(key)))


def shutdown() -> None:
    lib().prom_shutdown()


def pack_ternary(w: torch.Tensor, stream=None) -> torch.Tensor:
    """prom_pack_ternary: device int8 [cout, cin] -> device uint8 [cout, ceil(cin/4)]."""
    cout, cin = w.shape
    out = torch.empty((cout, (cin + 3) // 4), dtype=torch.uint8, device=w.device)
    _check(lib().prom_pack_ternary(_dev(w, torch.int8, "w"), cout, cin, out.data_ptr(),
                                   out.numel(), _stream(stream)), "prom_pack_ternary")
    return out


def quantize_ternary(w: torch.Tensor, want_alpha: bool = True, stream=None):
    """prom_quantize_ternary: device float32 [cout, cin] -> (packed uint8 [cout, ceil(cin/4)],
    alpha float32 [cout] or None)."""
    cout, cin = w.shape
    packed = torch.empty((cout, (cin + 3) // 4), dtype=torch.uint8, device=w.device)
    alpha = torch.empty((cout,), dtype=torch.float32, device=w.device) if want_alpha else None
    _check(lib().prom_quantize_ternary(_dev(w, torch.float32, "w"), cout, cin, packed.data_ptr(),
                                       packed.numel(), alpha.data_ptr() if want_alpha else None,
                                       _stream(stream)), "prom_quantize_ternary")
    return packed, alpha


class QuantizeJobs:
    """The job table of prom_quantize_ternary_batch for a list of device float32 [cout, cin] matrices,
    marshalled once (it holds raw pointers: the tensors are kept alive with it)."""

    def __init__(self, ws: Sequence[torch.Tensor], out=None):
        if out is None:
            out = [(torch.empty((w.shape[0], (w.shape[1] + 3) // 4), dtype=torch.uint8, device=w.device),
                    torch.empty((w.shape[0],), dtype=torch.float32, device=w.device)) for w in ws]
        self.ws, self.out, self.n = list(ws), out, len(ws)
        self.array = (PromQuantizeJob * self.n)()
        for j, (w, (packed, alpha)) in enumerate(zip(ws, out)):
            self.array[j] = PromQuantizeJob(_dev(w, torch.float32, "w"), w.shape[0], w.shape[1], packed.data_ptr(),
                                            packed.numel(), alpha.data_ptr())


def quantize_ternary_batch(ws: Optional[Sequence[torch.Tensor]] = None, out=None, stream=None,
                           jobs: Optional[QuantizeJobs] = None):
    """prom_quantize_ternary_batch: a list of device float32 [cout, cin] matrices -> a list of
    (packed uint8 [cout, ceil(cin/4)], alpha float32 [cout]); `out` may carry that list, `jobs` a
    table marshalled earlier (then ws and out are not looked at)."""
    if jobs is None:
        jobs = QuantizeJobs(ws, out)
    _check(lib().prom_quantize_ternary_batch(jobs.array, jobs.n, _stream(stream)), "prom_quantize_ternary_batch")
    return jobs.out


def requant_from_scale(scale: float):
    """prom_requant_from_scale: (mult, shift) for a real scale in (0, 1)."""
    m, s = C.c_int32(), C.c_int8()
    _check(lib().prom_requant_from_scale(float(scale), C.byref(m), C.byref(s)), "prom_requant_from_scale")
    return int(m.value), int(s.value)


def make_requant(bias: torch.Tensor, mult: torch.Tensor, shift: torch.Tensor,
                 act_min: int = 0, act_max: int = 127) -> PromRequant:
    rq = PromRequant(_dev(bias, torch.int32, "bias"), _dev(mult, torch.int32, "mult"),
                     _dev(shift, torch.int8, "shift"), int(act_min), int(act_max))
    rq._keep = (bias, mult, shift)      # the struct holds raw pointers: keep the tensors alive
    return rq


def pw_conv_i8(x: torch.Tensor, w_packed: torch.Tensor, cout: int, rq: PromRequant,
               y: Optional[torch.Tensor] = None, variant="auto", stream=None) -> torch.Tensor:
    """prom_pw_conv_i8 on device tensors; x is [m, cin] int8."""
    m, cin = x.shape
    if y is None:
        y = torch.empty((m, cout), dtype=torch.int8, device=x.device)
    _check(lib().prom_pw_conv_i8(_dev(x, torch.int8, "x"), m, cin,
                                 _dev(w_packed, torch.uint8, "w_packed"), cout, C.byref(rq),
                                 _dev(y, torch.int8, "y"), _variant(variant), _stream(stream)),
           "prom_pw_conv_i8")
    return y


def pw_prepare(m: int, cin: int, w_packed: torch.Tensor, cout: int, rq: PromRequant, stream=None):
    """prom_pw_prepare: the layer's prepared operands (a uint8 CUDA tensor), or None when the
    tensor-core variant cannot run the shape."""
    nbytes = int(lib().prom_pw_prepared_bytes(m, cin, cout))
    if nbytes == 0:
        return None
    buf = torch.empty((nbytes,), dtype=torch.uint8, device=w_packed.device)
    _check(lib().prom_pw_prepare(m, cin, _dev(w_packed, torch.uint8, "w_packed"), cout, C.byref(rq),
                                 buf.data_ptr(), nbytes, _stream(stream)), "prom_pw_prepare")
    return buf


def pw_conv_i8_prepared(x: torch.Tensor, cout: int, prepared: torch.Tensor, act_min: int = 0, act_max: int = 127,
                        y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """prom_pw_conv_i8_prepared on device tensors; x is [m, cin] int8."""
    m, cin = x.shape
    if y is None:
        y = torch.empty((m, cout), dtype=torch.int8, device=x.device)
    _check(lib().prom_pw_conv_i8_prepared(_dev(x, torch.int8, "x"), m, cin, cout,
                                          _dev(prepared, torch.uint8, "prepared"), act_min, act_max,
                                          _dev(y, torch.int8, "y"), _stream(stream)), "prom_pw_conv_i8_prepared")
    return y


def pw_conv_i8_res(x: torch.Tensor, w_packed: torch.Tensor, cout: int, rq: PromRequant,
                   res: torch.Tensor, y: Optional[torch.Tensor] = None, variant="auto",
                   stream=None) -> torch.Tensor:
    """prom_pw_conv_i8_res: the layer plus the int8 tensor `res` ([m, cout]) with saturation;
    pass y=res to form the sum in place."""
    m, cin = x.shape
    if tuple(res.shape) != (m, cout):
        raise ValueError("res must be [m, cout]")
    if y is None:
        y = torch.empty((m, cout), dtype=torch.int8, device=x.device)
    _check(lib().prom_pw_conv_i8_res(_dev(x, torch.int8, "x"), m, cin,
                                     _dev(w_packed, torch.uint8, "w_packed"), cout, C.byref(rq),
                                     _dev(res, torch.int8, "res"), _dev(y, torch.int8, "y"),
                                     _variant(variant), _stream(stream)),
           "prom_pw_conv_i8_res")
    return y


def pw_conv_i8_addsub_static(x: torch.Tensor, w_packed: torch.Tensor, cout: int, rq: PromRequant,
                             y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """prom_pw_conv_i8_addsub_static: the add/sub variant on the library's built-in
    scratch array, for callers that must not trigger a device allocation.  The
    output tensor is the caller's; pass `y` to keep this wrapper from allocating too."""
    m, cin = x.shape
    if y is None:
        y = torch.empty((m, cout), dtype=torch.int8, device=x.device)
    _check(lib().prom_pw_conv_i8_addsub_static(_dev(x, torch.int8, "x"), m, cin,
                                               _dev(w_packed, torch.uint8, "w_packed"), cout,
                                               C.byref(rq), _dev(y, torch.int8, "y"),
                                               _stream(stream)),
           "prom_pw_conv_i8_addsub_static")
    return y


def pw_conv_i8_acc32(x: torch.Tensor, w_packed: torch.Tensor, cout: int, stream=None) -> torch.Tensor:
    m, cin = x.shape
    acc = torch.empty((m, cout), dtype=torch.int32, device=x.device)
    _check(lib().prom_pw_conv_i8_acc32(_dev(x, torch.int8, "x"), m, cin,
                                       _dev(w_packed, torch.uint8, "w_packed"), cout,
                                       acc.data_ptr(), _stream(stream)), "prom_pw_conv_i8_acc32")
    return acc


def pw_conv_i8_host(x_host: torch.Tensor, w_packed: torch.Tensor, cout: int, rq: PromRequant,
                    y_host: torch.Tensor, workspace: torch.Tensor, variant="auto", stream=None):
    """prom_pw_conv_i8_host: host (pinned) activations in, host output out."""
    m, cin = x_host.shape
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("x_host / y_host must be host tensors")
    _check(lib().prom_pw_conv_i8_host(x_host.data_ptr(), m, cin,
                                      _dev(w_packed, torch.uint8, "w_packed"), cout, C.byref(rq),
                                      y_host.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                      _variant(variant), _stream(stream)), "prom_pw_conv_i8_host")
    return y_host


class LayerSeq:
    """A prom_layer array plus the tensors it points to (kept alive here)."""

    def __init__(self, layers: Sequence[dict], act_min: int = 0, act_max: int = 127):
        self.n = len(layers)
        self._keep: List[torch.Tensor] = []
        self.array = (PromLayer * self.n)()
        for i, l in enumerate(layers):
            for k in ("w_packed", "bias", "mult", "shift"):
                self._keep.append(l[k])
            self.array[i] = PromLayer(int(l["cin"]), int(l["cout"]), int(l["in_stride"]),
                                      _dev(l["w_packed"], torch.uint8, "w_packed"),
                                      make_requant(l["bias"], l["mult"], l["shift"],
                                                   int(l.get("act_min", act_min)),
                                                   int(l.get("act_max", act_max))))
            self.array[i].add_block_input = 1 if l.get("add_block_input") else 0
            if l.get("dw_w") is not None:
                # a real depthwise 3x3 in front: int8 [cin, 3, 3] weights and their constants
                for k in ("dw_w", "dw_bias", "dw_mult", "dw_shift"):
                    self._keep.append(l[k])
                self.array[i].dw_w = _dev(l["dw_w"], torch.int8, "dw_w")
                self.array[i].dw_rq = make_requant(l["dw_bias"], l["dw_mult"], l["dw_shift"], act_min, act_max)
        self.cout_last = int(layers[-1]["cout"])
        self.cin0 = int(layers[0]["cin"])
        self.total_stride = 1
        for l in layers:
            self.total_stride *= int(l["in_stride"])

    def workspace_bytes(self, batch: int, h0: int, w0: int) -> int:
        return int(lib().prom_layer_seq_workspace_bytes(self.array, self.n, batch, h0, w0))

    def host_workspace_bytes(self, batch: int, h0: int, w0: int) -> int:
        return int(lib().prom_layer_seq_host_workspace_bytes(self.array, self.n, batch, h0, w0))


def pw_layer_seq(seq: LayerSeq, x0: torch.Tensor, workspace: torch.Tensor,
                 y_out: Optional[torch.Tensor] = None, variant="auto", stream=None) -> torch.Tensor:
    """prom_pw_layer_seq on device tensors; x0 is [batch, h0, w0, cin0] int8."""
    batch, h0, w0, _ = x0.shape
    if y_out is None:
        y_out = torch.empty((batch, h0 // seq.total_stride, w0 // seq.total_stride, seq.cout_last),
                            dtype=torch.int8, device=x0.device)
    _check(lib().prom_pw_layer_seq(seq.array, seq.n, _dev(x0, torch.int8, "x0"), batch, h0, w0,
                                   workspace.data_ptr(), workspace.numel(),
                                   _dev(y_out, torch.int8, "y_out"), _variant(variant),
                                   _stream(stream)), "prom_pw_layer_seq")
    return y_out


def pw_layer_seq_host(seq: LayerSeq, x0_host: torch.Tensor, workspace: torch.Tensor,
                      y_out_host: torch.Tensor, variant="auto", stream=None) -> torch.Tensor:
    batch, h0, w0, _ = x0_host.shape
    if x0_host.is_cuda or y_out_host.is_cuda:
        raise ValueError("x0_host / y_out_host must be host tensors")
    _check(lib().prom_pw_layer_seq_host(seq.array, seq.n, x0_host.data_ptr(), batch, h0, w0,
                                        workspace.data_ptr(), workspace.numel(),
                                        y_out_host.data_ptr(), _variant(variant), _stream(stream)),
           "prom_pw_layer_seq_host")
    return y_out_host
