"""Helpers for the GPU parity tests: build one layer's inputs on the host (for
the oracle) and on the device (for the library) from the same seeded draws."""
import numpy as np
import torch

from paper_2505_03254_b200 import binding, synth


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


def run_variant(xd, wp, consts, cout, variant, act_min=0, act_max=127):
    rq = binding.make_requant(*consts, act_min, act_max)
    y = torch.full((xd.shape[0], cout), -77, dtype=torch.int8, device=xd.device)
    binding.pw_conv_i8(xd, wp, cout, rq, y=y, variant=variant)
    torch.cuda.synchronize()
    return y.cpu().numpy()


def first_mismatch(a, b):
    idx = np.argwhere(a != b)
    if len(idx) == 0:
        return None
    r, c = idx[0]
    return f"{len(idx)} mismatches, first at ({r},{c}): got {a[r, c]} want {b[r, c]}"
