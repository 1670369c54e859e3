"""Host logic of the tensor-core launch planner, exercised without a GPU (the plan query falls
back to a B200's nominal limits): every layer of the bench network and of its width variants
gets a plan, and every plan respects the limits the kernel relies on (tensor-memory columns,
shared memory, ring depths, divisibility of the folded problem, at most two CTAs per SM)."""
import pytest

from paper_2505_03254_b200 import binding, synth

SMS, SMEM_OPTIN = 148, 232448


def _check_plan(m, cin, cout, pl):
    fold, nt, groups, grid = pl["fold"], pl["nt"], pl["groups"], pl["grid"]
    assert fold in (1, 2, 4, 8) and m % fold == 0
    kf, nf = cin * fold, cout * fold
    assert kf % 16 == 0, "rows of the folded input are 16-byte multiples (tensor map)"
    assert nt % 8 == 0 and 8 <= nt <= 256 and nf % nt == 0
    n_sub = nf // nt
    assert n_sub % groups == 0 and grid % groups == 0 and 1 <= grid <= 2 * SMS
    if n_sub > 1:
        assert nt % 16 == 0 and nf % 16 == 0, "tensor-map stores need 16-byte rows"
    nt_pad = (nt + 15) // 16 * 16
    assert pl["nbuf"] in (2, 4) and pl["nbuf"] * nt_pad <= 512
    if grid > SMS:                       # two CTAs per SM share the 512 columns
        assert pl["nbuf"] * nt_pad <= 256 and 2 * pl["smem"] <= 233472 - 2048 + 2048
    assert 2 <= pl["stages"] <= 8
    assert pl["cw"] in (32, 64, 128) and (pl["cw"] >= min(kf, 128) or pl["cw"] == 128)
    assert 0 < pl["smem"] <= SMEM_OPTIN
    workers = grid // groups
    tiles = (m // fold + 127) // 128
    assert workers <= tiles, "no CTA without a tile"
    assert pl["est_us_x100"] > 0


@pytest.mark.parametrize("width", [0.75, 1.0, 1.4, 2.0])
@pytest.mark.parametrize("batch", [1, 8, 128])
def test_every_layer_gets_a_valid_plan(width, batch):
    binding.debug_tc_plan()
    seen = set()
    for l in synth.mobilenetv2_pointwise_layers(width=width):
        m = batch * l.h * l.w
        if (m, l.cin, l.cout) in seen:
            continue
        seen.add((m, l.cin, l.cout))
        pl = binding.debug_tc_plan_query(m, l.cin, l.cout)
        if pl is None:
            # the one documented refusal among these shapes: channel counts that are 8 modulo 16
            # need two rows folded into one, which an odd number of rows does not allow
            assert m % 2 == 1 and (l.cin % 16 or l.cout % 16), (m, l.cin, l.cout)
            continue
        _check_plan(m, l.cin, l.cout, pl)
        assert binding.debug_tc_plan_query(m, l.cin, l.cout) == pl      # cached, deterministic


def test_shapes_the_tensor_core_variant_refuses():
    binding.debug_tc_plan()
    assert binding.debug_tc_plan_query(1000, 12, 64) is None          # cin not a multiple of 8
    assert binding.debug_tc_plan_query(1000, 64, 20) is None          # cout not a multiple of 8
    assert binding.debug_tc_plan_query(0, 64, 64) is None             # nothing to do
    assert binding.debug_tc_plan_query(129, 24, 24) is None           # odd rows, rows not 16-byte multiples


def test_forced_plans_are_honoured_or_refused():
    try:
        binding.debug_tc_plan(1, 32, 2, 2, 0)
        pl = binding.debug_tc_plan_query(25088, 64, 384)
        assert pl is not None and (pl["fold"], pl["nt"], pl["groups"]) == (1, 32, 2)
        _check_plan(25088, 64, 384, pl)
        binding.debug_tc_plan(1, 96, 1, 4, 0)                          # three CTAs per SM: 2 x 96 columns > 128
        assert binding.debug_tc_plan_query(1605632, 16, 96) is None
        binding.debug_tc_plan(1, 48, 1, 4, 0)
        pl = binding.debug_tc_plan_query(1605632, 16, 96)
        assert pl is not None and pl["grid"] == 3 * SMS and pl["smem"] <= (233472 - 3 * 1024) // 3
    finally:
        binding.debug_tc_plan()
