"""Helpers for the GPU parity tests: build one layer's inputs on the host (for
the oracle) and on the device (for the library) from the same seeded draws,
and give every buffer the library writes a band of canary bytes on both sides."""
import numpy as np
import torch

from paper_2505_03254_b200 import binding, synth

GUARD = 4096          # canary bytes before and after a guarded buffer
CANARY = 0x5A


class Guarded:
    """A device buffer of `nbytes` bytes (dtype int8 or uint8) with GUARD canary
    bytes on either side: a store that strays past the buffer's ends shows up
    in check()."""

    def __init__(self, nbytes, dtype=torch.int8, fill=-77, device="cuda"):
        self.nbytes = int(nbytes)
        self.raw = torch.full((self.nbytes + 2 * GUARD,), CANARY, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD:GUARD + self.nbytes].view(dtype)
        if self.nbytes:
            self.t.fill_(fill)

    def view(self, *shape):
        return self.t.view(*shape)

    def check(self, what="buffer"):
        torch.cuda.synchronize()
        lo = self.raw[:GUARD]
        hi = self.raw[GUARD + self.nbytes:]
        assert bool((lo == CANARY).all()), f"{what}: bytes written before its start"
        assert bool((hi == CANARY).all()), f"{what}: bytes written past its end"


def make_case(seed, m, cin, cout, zero_frac=0.5, act="i8", shift_lo=None, shift_hi=None):
    if act == "i8":
        x = synth.act_uniform_i8(seed, (m, cin))
    elif act == "relu6":
        x = synth.act_post_relu6(seed, (m, cin))
    else:
        x = synth.act_uniform_0_127(seed, (m, cin))
    lay = synth.make_layer(seed, cin, cout, zero_frac)
    if shift_lo is not None:
        g = torch.Generator().manual_seed(seed)
        lay["shift"] = torch.randint(shift_lo, shift_hi + 1, (cout,), generator=g).to(torch.int8)
    return x, lay


def to_device(x, lay, dev="cuda"):
    xd = x.to(dev)
    wp = binding.pack_ternary(lay["w"].to(dev))
    bias, mult, shift = lay["bias"].to(dev), lay["mult"].to(dev), lay["shift"].to(dev)
    return xd, wp, (bias, mult, shift)


def oracle_y(oracle, x, lay, act_min=0, act_max=127):
    return oracle.conv_mul(x.numpy(), lay["w"].numpy(), lay["bias"].numpy(), lay["mult"].numpy(),
                           lay["shift"].numpy(), act_min, act_max)


def run_variant_device(xd, wp, consts, cout, variant, act_min=0, act_max=127):
    """One call into a guarded output; returns the device tensor (guards checked)."""
    rq = binding.make_requant(*consts, act_min, act_max)
    g = Guarded(xd.shape[0] * cout)
    y = g.view(xd.shape[0], cout)
    binding.pw_conv_i8(xd, wp, cout, rq, y=y, variant=variant)
    g.check(f"output of variant {variant}")
    return y


def run_variant(xd, wp, consts, cout, variant, act_min=0, act_max=127):
    return run_variant_device(xd, wp, consts, cout, variant, act_min, act_max).cpu().numpy()


def first_mismatch(a, b):
    idx = np.argwhere(a != b)
    if len(idx) == 0:
        return None
    r, c = idx[0]
    return f"{len(idx)} mismatches, first at ({r},{c}): got {a[r, c]} want {b[r, c]}"


def sample_rows(m, tile=128, edge=512, one_in=64, seed=0):
    """Rows of an m-row matrix on which the oracle checks a large launch: the first and
    last `edge` rows, the two rows on either side of every `tile`-row boundary, and a hashed
    1/`one_in` of the rest.  Rows are independent units of the computation, so the sampled
    rows are checked exactly."""
    if m <= 2 * edge + 2 * tile:
        return np.arange(m, dtype=np.int64)
    keep = np.zeros(m, dtype=bool)
    keep[:edge] = True
    keep[m - edge:] = True
    b = np.arange(tile, m, tile, dtype=np.int64)
    keep[b] = True
    keep[b - 1] = True
    h = synth.hash64(seed, 77, 0, m).numpy().astype(np.uint64)
    keep |= (h % np.uint64(one_in)) == 0
    return np.nonzero(keep)[0].astype(np.int64)
