"""GPU parity of prom_quantize_act_absmax (paper Eq. 6-7) with the CPU oracle: codes, gamma
and scale bit for bit (both sides take the decision in binary32 with the same two correctly
rounded operations), on the staged cluster route, the re-reading cluster route and the
two-kernel route, ragged sizes included."""
import numpy as np
import pytest
import torch

from paper_2505_03254_b200 import binding

pytestmark = pytest.mark.gpu


def _input(seed, shape, spread=True):
    """Seeded float32 activations: PReLU-like outputs (negative side scaled down), a different
    magnitude per sample, a share of exact zeros and of values sitting exactly on rounding ties."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(shape).astype(np.float32)
    x = np.where(x < 0, x * np.float32(0.25), x)
    x[rng.random(shape) < 0.2] = 0.0
    if spread:
        mags = np.float32(2.0) ** rng.integers(-12, 12, size=(shape[0],) + (1,) * (len(shape) - 1))
        x = x * mags.astype(np.float32)
    return x


def _check(oracle, x):
    want_q, want_g, want_s = oracle.quantize_act_absmax(x)
    q, g, s = binding.quantize_act_absmax(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    assert binding.last_device_status() == binding.PROM_OK
    assert np.array_equal(g.cpu().numpy().view(np.uint32), want_g.view(np.uint32))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    got = q.cpu().numpy()
    bad = np.argwhere(got != want_q)
    assert len(bad) == 0, (bad[:5].tolist(), got[tuple(bad[0])], want_q[tuple(bad[0])])


@pytest.mark.parametrize("shape", [
    (3, 16),                   # one 16-float piece per sample, cluster of 1
    (4, 14, 14, 64),           # 12 544 per sample: one CTA
    (2, 56, 56, 24),           # 75 264: a cluster of 2
    (2, 112, 112, 16),         # 200 704: a cluster of 4, ragged last slices
    (3, 112, 112, 32),         # 401 408: a cluster of 8, the bench's input tensor shape
])
def test_fused_route(oracle, shape):
    _check(oracle, _input(11, shape))


@pytest.mark.parametrize("shape", [
    (5, 7),                    # not a multiple of 16: two kernels (maxima, then codes)
    (3, 1001),
    (2, 7, 7, 1280 + 8),
    (2, 160, 160, 24),         # 614 400 per sample: too large for a cluster's shared memory,
    (3, 224, 224, 16),         # 802 816: the clusters read their slices twice instead
])
def test_other_routes(oracle, shape):
    _check(oracle, _input(12, shape))


def test_ties_zero_samples_and_exact_integers(oracle):
    x = np.zeros((4, 64), dtype=np.float32)
    x[1, :8] = [127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5]           # scale 1: ties to even
    x[2, :4] = [5e-6, -2e-6, 1e-6, 0.0]                                   # below eps
    x[3] = np.arange(-32, 32, dtype=np.float32) * 4 - 1                   # integers, max |x| = 129
    _check(oracle, x)
    q, g, s = binding.quantize_act_absmax(torch.from_numpy(x).cuda())
    assert q[1, :8].tolist() == [127, 0, 2, 2, 0, -2, -2, 126]
    assert not q[0].any().item()


def test_repeated_calls_and_empty_batch(oracle):
    x = _input(13, (2, 28, 28, 96))
    for _ in range(3):
        _check(oracle, x)
    e = torch.empty((0, 16), dtype=torch.float32, device="cuda")
    q, g, s = binding.quantize_act_absmax(e)
    assert q.shape == (0, 16) and g.numel() == 0


def test_seeded_shape_fuzz(oracle):
    """Random batch sizes and sample sizes across all three routes (multiples of 16 small and
    large, and sizes that are not)."""
    rng = np.random.default_rng(97)
    for case in range(20):
        batch = int(rng.integers(1, 40))
        kind = case % 3
        if kind == 0:
            per = 16 * int(rng.integers(1, 4000))
        elif kind == 1:
            per = int(rng.integers(1, 50000))
        else:
            per = 16 * int(rng.integers(30000, 60000))          # beyond a cluster's shared memory
            batch = min(batch, 4)
        _check(oracle, _input(300 + case, (batch, per)))
