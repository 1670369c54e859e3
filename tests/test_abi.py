"""The C-ABI library loads without a GPU, exports every symbol the header
declares, and rejects bad arguments on the host before touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2505_03254_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    import glob
    names = set()
    for path in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = open(path).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(prom_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "prom_pack_ternary" in names and "prom_pw_conv_i8" in names and "prom_pw_layer_seq" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_packed_bytes(lib):
    assert binding.packed_bytes(384, 64) == 384 * 16
    assert binding.packed_bytes(3, 6) == 6
    assert binding.packed_bytes(1, 1) == 1
    assert binding.packed_bytes(-1, 4) == 0


def test_status_strings(lib):
    seen = {binding.status_string(i) for i in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert binding.status_string(99) == "unknown status"


def test_host_side_argument_checks(lib):
    rq = binding.PromRequant(16, 16, 16, 0, 127)
    A = 0x1000  # a 16-byte-aligned non-null address; never dereferenced by these calls
    st = None
    f = lib.prom_pw_conv_i8
    assert f(None, 4, 8, A, 8, C.byref(rq), A, 0, st) == binding.PROM_ERR_NULL
    assert f(A, 4, 8, A, 8, None, A, 0, st) == binding.PROM_ERR_NULL
    assert f(A, -1, 8, A, 8, C.byref(rq), A, 0, st) == binding.PROM_ERR_SHAPE
    assert f(A, 4, 0, A, 8, C.byref(rq), A, 0, st) == binding.PROM_ERR_SHAPE
    assert f(A, 4, 8, A, 5000, C.byref(rq), A, 0, st) == binding.PROM_ERR_SHAPE
    assert f(A + 4, 4, 8, A, 8, C.byref(rq), A, 0, st) == binding.PROM_ERR_ALIGN
    bad = binding.PromRequant(16, 16, 16, 5, 4)
    assert f(A, 4, 8, A, 8, C.byref(bad), A, 0, st) == binding.PROM_ERR_BAD_REQUANT
    bad = binding.PromRequant(16, 16, 16, -129, 4)
    assert f(A, 4, 8, A, 8, C.byref(bad), A, 0, st) == binding.PROM_ERR_BAD_REQUANT
    bad = binding.PromRequant(0, 16, 16, 0, 127)
    assert f(A, 4, 8, A, 8, C.byref(bad), A, 0, st) == binding.PROM_ERR_NULL
    # m == 0 is a no-op
    assert f(A, 0, 8, A, 8, C.byref(rq), A, 0, st) == binding.PROM_OK
    assert lib.prom_pack_ternary(None, 4, 4, A, 4, st) == binding.PROM_ERR_NULL
    assert lib.prom_pack_ternary(A, 4, 4, A, 3, st) == binding.PROM_ERR_WORKSPACE
    assert lib.prom_pack_ternary(A, 0, 4, A, 3, st) == binding.PROM_ERR_SHAPE


def test_layer_seq_shape_checks(lib):
    L = binding.PromLayer
    rq = binding.PromRequant(16, 16, 16, 0, 127)
    arr = (L * 3)(L(8, 16, 1, 16, rq), L(16, 8, 2, 16, rq), L(8, 24, 1, 16, rq))
    ws = lib.prom_layer_seq_workspace_bytes(arr, 3, 2, 8, 8)
    # region A holds layer 0's output (2*8*8*16), region B layer 1's (2*4*4*8), each 256-rounded
    assert ws == 2048 + 256
    assert lib.prom_layer_seq_host_workspace_bytes(arr, 3, 2, 8, 8) == ws + 1024 + 768
    arr[1].cin = 12          # does not chain
    assert lib.prom_layer_seq_workspace_bytes(arr, 3, 2, 8, 8) == 0
    arr[1].cin = 16
    assert lib.prom_layer_seq_workspace_bytes(arr, 3, 2, 7, 8) == 0   # odd size under stride 2
    A = 0x1000
    assert lib.prom_pw_layer_seq(arr, 3, A, 2, 7, 8, A, 1 << 20, A, 0, None) == binding.PROM_ERR_SHAPE
    assert lib.prom_pw_layer_seq(arr, 3, A, 2, 8, 8, A, 16, A, 0, None) == binding.PROM_ERR_WORKSPACE
    assert lib.prom_pw_layer_seq(arr, 3, None, 2, 8, 8, A, 1 << 20, A, 0, None) == binding.PROM_ERR_NULL


def test_requant_from_scale_matches_the_oracle(lib, oracle):
    """Host-only helper: same (mult, shift) as the oracle's definition on random and
    boundary scales, and the documented refusals."""
    import numpy as np
    rng = np.random.default_rng(5)
    scales = list(2.0 ** rng.uniform(-31.9, -0.001, size=3000))
    scales += [0.5, 0.25, 2.0 ** -32 * 1.5, 2.0 ** -13, (1 - 2.0 ** -33) * 2.0 ** -9]
    for sc in scales:
        assert binding.requant_from_scale(sc) == oracle.requant_from_scale(sc), sc
    # refused by both: not positive, not below one, rounding up to one, or too small for shift 31
    for bad in (0.0, -0.5, 1.0, 7.0, 1 - 2.0 ** -40, 2.0 ** -40, float("nan")):
        with pytest.raises(binding.PromError) as e:
            binding.requant_from_scale(bad)
        assert e.value.code == binding.PROM_ERR_BAD_REQUANT
        with pytest.raises(ValueError):
            oracle.requant_from_scale(bad)


def test_attributes_are_recorded_per_device(lib):
    """The table behind the per-device kernel attributes (a kernel's shared-memory limit
    belongs to the device that was current when it was raised): each (device, kernel) pair is
    new exactly once, whatever the order of the calls."""
    assert binding.debug_once_per_device(0, 11)
    assert not binding.debug_once_per_device(0, 11)
    assert binding.debug_once_per_device(1, 11)          # the same kernel on a second device
    assert binding.debug_once_per_device(0, 12)          # another kernel on the first
    assert not binding.debug_once_per_device(1, 11)
    assert not binding.debug_once_per_device(0, 12)
