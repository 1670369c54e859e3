"""Failure detection and per-device bookkeeping on a GPU, in their harmless forms: a bounded
device-side wait that is left to run out must give up by itself and surface as
PROM_ERR_TIMEOUT; nothing here traps, faults or waits without a limit."""
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


def test_a_wait_that_nothing_ends_gives_up_and_is_reported(oracle):
    assert binding.last_device_status() == binding.PROM_OK
    assert binding.debug_wait_timeout(5000) == 1          # the library's wait_bar returned false
    assert binding.last_device_status() == binding.PROM_ERR_TIMEOUT
    assert binding.last_device_status() == binding.PROM_OK   # reading clears the word
    # the context is as usable as before
    x, lay = make_case(71, 300, 64, 96)
    got = run_variant(*to_device(x, lay), 96, "tc")
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


def test_limit_outside_the_documented_range_is_refused():
    for bad in (0, 999, 100_000_001):
        rc = binding.lib().prom_debug_wait_timeout(bad, None, None)
        assert rc == binding.PROM_ERR_SHAPE


def test_setting_the_device_again_keeps_large_launches_working(oracle):
    """Kernels that need more than 48 KB of dynamic shared memory after the current device has
    been selected a second time (the attribute table is keyed by device)."""
    torch.cuda.set_device(0)
    x, lay = make_case(72, 260, 960, 160)
    xd, wp, consts = to_device(x, lay)
    want = oracle_y(oracle, x, lay)
    for _ in range(2):
        torch.cuda.set_device(0)
        for variant in ("tc", "addsub"):
            assert first_mismatch(run_variant(xd, wp, consts, 160, variant), want) is None


def test_bad_constants_leave_the_affected_outputs_unwritten():
    """A channel whose constants are out of range: status word set, and the add/sub variant
    leaves that channel's bytes untouched whether Cout is a multiple of four or not."""
    for cout in (16, 18):
        x, lay = make_case(73, 64, 16, cout)
        lay["shift"][3] = 40
        xd, wp, consts = to_device(x, lay)
        y = run_variant(xd, wp, consts, cout, "addsub")
        assert binding.last_device_status() == binding.PROM_ERR_BAD_REQUANT
        assert (y[:, 3] == -77).all(), cout
        assert (y[:, 4] != -77).any(), cout
