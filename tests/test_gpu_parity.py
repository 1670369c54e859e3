"""GPU parity: every variant of the library against the CPU oracle, byte for
byte, through the C ABI."""
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


def test_pack_matches_oracle(oracle):
    for seed, (cout, cin) in enumerate([(1, 1), (5, 3), (16, 24), (37, 145), (384, 64), (1280, 320)]):
        w = synth.ternary_weights(seed, cout, cin, 0.5)
        got = binding.pack_ternary(w.cuda()).cpu().numpy()
        assert np.array_equal(got, oracle.pack(w.numpy()))


def test_pack_rejects_invalid_weights():
    w = torch.zeros((4, 8), dtype=torch.int8)
    w[2, 5] = 2
    with pytest.raises(binding.PromError) as e:
        binding.pack_ternary(w.cuda())
    assert e.value.code == binding.PROM_ERR_BAD_WEIGHT


def test_acc32_matches_oracle(oracle):
    x, lay = make_case(3, 77, 40, 24)
    xd, wp, _ = to_device(x, lay)
    acc = binding.pw_conv_i8_acc32(xd, wp, 24).cpu().numpy()
    _, want = oracle.conv_mul(x.numpy(), lay["w"].numpy(), lay["bias"].numpy(), lay["mult"].numpy(),
                              lay["shift"].numpy(), want_acc=True)
    assert np.array_equal(acc, want)


# (m, cin, cout): several tiles and a ragged tail, odd channel counts included
NAIVE_SHAPES = [(1, 1, 1), (196, 64, 384), (300, 24, 144), (129, 7, 5), (1000, 145, 37)]
TC_SHAPES = [(196, 64, 384), (1, 16, 16), (127, 16, 96), (128, 32, 16), (129, 96, 24),
             (1000, 144, 32), (777, 192, 64), (515, 384, 96), (300, 576, 160), (260, 960, 320),
             (333, 320, 1280), (2000, 16, 96), (386, 24, 144), (258, 144, 24), (130, 40, 8),
             (4100, 64, 384), (200, 160, 960), (131, 960, 160), (64, 8, 8), (50000, 32, 192)]
SMALLK_SHAPES = [(196, 64, 384), (1000, 16, 96), (129, 24, 144), (333, 4, 3), (500, 32, 16), (77, 60, 10)]
ADDSUB_SHAPES = [(196, 64, 384), (1000, 16, 96), (129, 24, 144), (300, 145, 37), (260, 960, 320),
                 (131, 600, 9)]


@pytest.mark.parametrize("m,cin,cout", NAIVE_SHAPES)
def test_naive(oracle, m, cin, cout):
    x, lay = make_case(10, m, cin, cout)
    got = run_variant(*to_device(x, lay), cout, "naive")
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


@pytest.mark.parametrize("m,cin,cout", TC_SHAPES)
def test_tc(oracle, m, cin, cout):
    x, lay = make_case(11, m, cin, cout)
    got = run_variant(*to_device(x, lay), cout, "tc")
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


@pytest.mark.parametrize("m,cin,cout", SMALLK_SHAPES)
def test_smallk(oracle, m, cin, cout):
    x, lay = make_case(12, m, cin, cout)
    got = run_variant(*to_device(x, lay), cout, "smallk")
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


@pytest.mark.parametrize("m,cin,cout", ADDSUB_SHAPES)
@pytest.mark.parametrize("zero_frac", [0.3, 0.9])
def test_addsub(oracle, m, cin, cout, zero_frac):
    x, lay = make_case(13, m, cin, cout, zero_frac)
    got = run_variant(*to_device(x, lay), cout, "addsub")
    assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


@pytest.mark.parametrize("variant", ["naive", "tc", "smallk", "addsub", "auto"])
def test_signed_clamp_and_wide_shifts(oracle, variant):
    """act_min < 0 pins the rounding of negative values; shifts 0..20 leave the
    tensor-core variant's fast epilogue."""
    x, lay = make_case(14, 517, 32, 48, shift_lo=0, shift_hi=20)
    xd, wp, consts = to_device(x, lay)
    for lo, hi in [(-128, 127), (-5, 90), (0, 127), (3, 100)]:
        got = run_variant(xd, wp, consts, 48, variant, lo, hi)
        assert first_mismatch(got, oracle_y(oracle, x, lay, lo, hi)) is None


@pytest.mark.parametrize("variant", ["tc", "smallk", "addsub", "naive"])
def test_ties_on_device(oracle, variant):
    """mult = 2^30, shift = 0, bias = 0: every odd accumulator is a tie."""
    m, cin, cout = 256, 16, 16
    x = synth.act_uniform_i8(15, (m, cin))
    lay = synth.make_layer(15, cin, cout, 0.5)
    lay["bias"] = torch.zeros(cout, dtype=torch.int32)
    lay["mult"] = torch.full((cout,), 1 << 30, dtype=torch.int32)
    lay["shift"] = torch.zeros(cout, dtype=torch.int8)
    xd, wp, consts = to_device(x, lay)
    for lo, hi in [(-128, 127), (0, 127)]:
        got = run_variant(xd, wp, consts, cout, variant, lo, hi)
        assert first_mismatch(got, oracle_y(oracle, x, lay, lo, hi)) is None


@pytest.mark.parametrize("variant", ["tc", "naive"])
def test_small_negative_ties_with_the_full_int8_clamp(oracle, variant):
    """One-hot weight rows (an output is +-1 times one input value, plus a small bias) with
    mult = 2^30 and shifts 0..4: outputs inside [-128, 127] that sit on ties of either sign,
    which round away from zero."""
    m, cin, cout = 512, 32, 32
    x = synth.act_uniform_i8(19, (m, cin))
    lay = synth.make_layer(19, cin, cout, 0.5)
    w = torch.zeros((cout, cin), dtype=torch.int8)
    for o in range(cout):
        w[o, (5 * o) % cin] = 1 if o % 3 else -1
    lay["w"] = w
    lay["bias"] = (torch.arange(cout, dtype=torch.int32) % 5) - 2
    lay["mult"] = torch.full((cout,), 1 << 30, dtype=torch.int32)
    lay["shift"] = (torch.arange(cout) % 5).to(torch.int8)
    xd, wp, consts = to_device(x, lay)
    want = oracle_y(oracle, x, lay, -128, 127)
    t = (x.numpy().astype(np.int64) @ w.numpy().T.astype(np.int64)) + lay["bias"].numpy()
    sh = lay["shift"].numpy().astype(np.int64) + 1
    ties = (t % (1 << sh)) == (1 << (sh - 1))
    assert (ties & (t < 0)).sum() > 100 and (ties & (t > 0)).sum() > 100
    assert np.array_equal(want[ties], (np.sign(t) * ((np.abs(t) + (1 << (sh - 1))) >> sh))[ties])
    got = run_variant(xd, wp, consts, cout, variant, -128, 127)
    assert first_mismatch(got, want) is None


def test_extreme_values(oracle):
    """All activations -128 against all +1 / all -1 weights at Cin = 960."""
    m, cin, cout = 130, 960, 16
    x = torch.full((m, cin), -128, dtype=torch.int8)
    lay = synth.make_layer(16, cin, cout, 0.0)
    lay["w"][:8] = 1
    lay["w"][8:] = -1
    xd, wp, consts = to_device(x, lay)
    for variant in ["tc", "addsub", "naive"]:
        for lo, hi in [(0, 127), (-128, 127)]:
            got = run_variant(xd, wp, consts, cout, variant, lo, hi)
            assert first_mismatch(got, oracle_y(oracle, x, lay, lo, hi)) is None


def test_bad_constants_are_reported():
    x, lay = make_case(17, 64, 16, 16)
    lay["shift"][3] = 40
    xd, wp, consts = to_device(x, lay)
    for variant in ["naive", "tc", "smallk", "addsub"]:
        run_variant(xd, wp, consts, 16, variant)
        assert binding.last_device_status() == binding.PROM_ERR_BAD_REQUANT
    assert binding.last_device_status() == binding.PROM_OK


def test_invalid_code_is_reported():
    x, lay = make_case(18, 64, 16, 16)
    xd, wp, consts = to_device(x, lay)
    wp[2, 1] = 0b00100000          # code 10 in the third slot
    for variant in ["naive", "tc", "smallk", "addsub"]:
        run_variant(xd, wp, consts, 16, variant)
        assert binding.last_device_status() == binding.PROM_ERR_BAD_WEIGHT


def test_unsupported_shapes_are_refused():
    x, lay = make_case(19, 65, 20, 12)
    xd, wp, consts = to_device(x, lay)
    rq = binding.make_requant(*consts)
    for variant in ["tc"]:
        with pytest.raises(binding.PromError) as e:
            binding.pw_conv_i8(xd, wp, 12, rq, variant=variant)
        assert e.value.code == binding.PROM_ERR_UNSUPPORTED
    x, lay = make_case(19, 64, 128, 12)
    xd, wp, consts = to_device(x, lay)
    with pytest.raises(binding.PromError) as e:
        binding.pw_conv_i8(xd, wp, 12, binding.make_requant(*consts), variant="smallk")
    assert e.value.code == binding.PROM_ERR_UNSUPPORTED


def test_auto_handles_any_shape(oracle):
    for m, cin, cout in [(65, 20, 12), (33, 7, 5), (131, 24, 144), (100, 2000, 8)]:
        x, lay = make_case(20, m, cin, cout)
        got = run_variant(*to_device(x, lay), cout, "auto")
        assert first_mismatch(got, oracle_y(oracle, x, lay)) is None


def test_host_buffer_entry_point(oracle):
    m, cin, cout = 700, 64, 96
    x, lay = make_case(21, m, cin, cout)
    _, wp, consts = to_device(x, lay)
    rq = binding.make_requant(*consts)
    xh = x.pin_memory()
    yh = torch.empty((m, cout), dtype=torch.int8).pin_memory()
    ws = torch.empty(((m * cin + 255) // 256 * 256 + (m * cout + 255) // 256 * 256,),
                     dtype=torch.uint8, device="cuda")
    binding.pw_conv_i8_host(xh, wp, cout, rq, yh, ws)
    torch.cuda.synchronize()
    assert first_mismatch(yh.numpy(), oracle_y(oracle, x, lay)) is None


def test_empty_and_single_row(oracle):
    """m = 0 is a no-op that touches nothing; m = 1 and m = 2 are the smallest tiles."""
    x, lay = make_case(22, 4, 32, 48)
    xd, wp, consts = to_device(x, lay)
    rq = binding.make_requant(*consts)
    y = torch.full((0, 48), 7, dtype=torch.int8, device="cuda")
    for variant in ["auto", "tc", "smallk", "addsub", "naive"]:
        binding.pw_conv_i8(xd[:0], wp, 48, rq, y=y, variant=variant)
    for rows in (1, 2):
        want = oracle_y(oracle, x[:rows], lay)
        for variant in ["auto", "smallk", "addsub", "naive"]:
            got = run_variant(xd[:rows].contiguous(), wp, consts, 48, variant)
            assert first_mismatch(got, want) is None, (rows, variant)


def test_largest_channel_counts(oracle):
    """Cin = Cout = 4096, the largest the interface accepts (weights 16 M ternary values)."""
    m, c = 260, 4096
    x = synth.act_uniform_i8(23, (m, c))
    lay = synth.make_layer(23, c, c, 0.5)
    xd, wp, consts = to_device(x, lay)
    rows = np.array([0, 1, 127, 128, 129, 259])
    want = oracle_y(oracle, x[rows], lay)
    ref = None
    for variant in ["tc", "naive"]:
        got = run_variant(xd, wp, consts, c, variant)
        assert first_mismatch(got[rows], want) is None, variant
        if ref is None:
            ref = got
        else:
            assert np.array_equal(got, ref)


def test_seeded_shape_fuzz(oracle):
    """Sixty seeded random shapes (rows 1..5000, channel counts multiples of 8 up to 640, both
    clamps, a shift span that forces either epilogue) through AUTO and, where it accepts the
    shape, the tensor-core variant: the planner's corner cases rather than the network's shapes."""
    rng = np.random.default_rng(4242)
    for case in range(60):
        m = int(rng.integers(1, 5001))
        cin = 8 * int(rng.integers(1, 81))
        cout = 8 * int(rng.integers(1, 81))
        x = synth.act_uniform_i8(900 + case, (m, cin)) if case % 2 else synth.act_uniform_0_127(900 + case, (m, cin))
        lay = synth.make_layer(900 + case, cin, cout, float(rng.choice([0.3, 0.5, 0.9])))
        shift = lay["shift"].numpy().copy()
        if case % 3 == 0:
            shift[: max(1, cout // 4)] = 2            # a shift span above 4: the exact epilogue
        lo, hi = (0, 127) if case % 4 else (-128, 127)
        want = oracle.conv_mul(x.numpy(), lay["w"].numpy(), lay["bias"].numpy(), lay["mult"].numpy(), shift,
                               act_min=lo, act_max=hi)
        wp = binding.pack_ternary(lay["w"].cuda())
        rq = binding.make_requant(lay["bias"].cuda(), lay["mult"].cuda(), torch.from_numpy(shift).cuda(),
                                  act_min=lo, act_max=hi)
        for variant in ("auto", "tc"):
            try:
                y = binding.pw_conv_i8(x.cuda(), wp, cout, rq, variant=variant)
            except binding.PromError as e:
                assert variant == "tc" and e.code == binding.PROM_ERR_UNSUPPORTED, (case, m, cin, cout, variant, e)
                continue
            torch.cuda.synchronize()
            assert binding.last_device_status() == binding.PROM_OK, (case, m, cin, cout, variant)
            bad = np.argwhere(y.cpu().numpy() != want)
            assert len(bad) == 0, (case, m, cin, cout, variant, lo, hi, bad[:3].tolist())


@pytest.mark.parametrize("m,cin,cout", TC_SHAPES)
def test_tc_from_prepared_operands(oracle, m, cin, cout):
    """The operands written once by prom_pw_prepare, then two calls from them."""
    x, lay = make_case(24, m, cin, cout)
    xd, wp, consts = to_device(x, lay)
    want = oracle_y(oracle, x, lay)
    prep = binding.pw_prepare(m, cin, wp, cout, binding.make_requant(*consts))
    assert prep is not None and prep.numel() == binding.lib().prom_pw_prepared_bytes(m, cin, cout)
    for _ in range(2):
        y = torch.full((m, cout), -77, dtype=torch.int8, device="cuda")
        binding.pw_conv_i8_prepared(xd, cout, prep, y=y)
        torch.cuda.synchronize()
        assert first_mismatch(y.cpu().numpy(), want) is None


def test_prepared_operands_clamps_and_refusals(oracle):
    m, cin, cout = 517, 64, 48
    x, lay = make_case(25, m, cin, cout, shift_lo=0, shift_hi=20)
    xd, wp, consts = to_device(x, lay)
    for lo, hi in [(-128, 127), (0, 127), (-5, 90)]:
        prep = binding.pw_prepare(m, cin, wp, cout, binding.make_requant(*consts, lo, hi))
        y = binding.pw_conv_i8_prepared(xd, cout, prep, lo, hi)
        torch.cuda.synchronize()
        assert first_mismatch(y.cpu().numpy(), oracle_y(oracle, x, lay, lo, hi)) is None, (lo, hi)
    # operands prepared for one clamp, call made with another: refused on the device
    y = torch.full((m, cout), -77, dtype=torch.int8, device="cuda")
    binding.pw_conv_i8_prepared(xd, cout, prep, 0, 127, y=y)
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_ERR_BAD_REQUANT
    assert bool((y == -77).all())
    # shapes the tensor-core variant cannot run have no prepared form
    assert binding.lib().prom_pw_prepared_bytes(65, 20, 12) == 0
    assert binding.pw_prepare(65, 20, wp, 12, binding.make_requant(*consts)) is None
    rc = binding.lib().prom_pw_prepare(65, 20, wp.data_ptr(), 12, binding.make_requant(*consts), wp.data_ptr(), 1 << 20, None)
    assert rc == binding.PROM_ERR_UNSUPPORTED
    # too small a buffer
    small = torch.empty((256,), dtype=torch.uint8, device="cuda")
    rc = binding.lib().prom_pw_prepare(m, cin, wp.data_ptr(), cout, binding.make_requant(*consts), small.data_ptr(), 256, None)
    assert rc == binding.PROM_ERR_WORKSPACE
