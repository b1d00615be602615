"""Pins for block-scaled rounding (Section I-A: blocks with a power-of-two scale)."""
import numpy as np
import pytest

from oracle import capi
from helpers import FMTS, bits_f32, random_f32, edge_values_f32

EMAX = {"bf16": 127, "fp16": 15, "e4m3": 8, "e5m2": 15}


@pytest.mark.parametrize("fmt", FMTS)
def test_block_scaled_is_per_block_power_of_two_scaling(fmt):
    """Scale bytes from numpy's frexp of the block maximum; codes equal plain rounding of x * 2^-e
    with the same global indices."""
    rng = np.random.default_rng(50)
    n = 32 * 40 + 13
    x = bits_f32(random_f32(rng, n, -30, 20))
    x[:64] *= 0.0                                   # an all-zero block and a block starting with zeros
    x[70] = np.inf; x[71] = np.nan                  # specials do not set the scale
    x[96:128] = bits_f32(edge_values_f32()[:32])
    codes, scales = capi.fbsr_round_mx(x, fmt, "srf", 3, seed=8, offset=5)
    for b in range(len(scales)):
        blk = x[32 * b: 32 * b + 32]
        fin = np.abs(blk[np.isfinite(blk)])
        amax = fin.max() if fin.size else 0.0
        e = -127
        if amax >= 2.0 ** -126:
            e = int(np.clip(np.frexp(np.float64(amax))[1] - 1 - EMAX[fmt], -127, 127))
        assert scales[b] == e + 127
        y = (blk.astype(np.float64) * 2.0 ** -e).astype(np.float32)     # exact scaling, one rounding when subnormal
        expect = capi.fbsr_round(y, fmt, "srf", 3, seed=8, offset=5 + 32 * b)
        ok = ~np.isnan(blk)
        assert np.array_equal(codes[32 * b: 32 * b + 32][ok], expect[ok])
        # the block maximum lands in the top binade of the format (or saturates to M)
        if fin.size and amax >= 2.0 ** -100 and amax * 2.0 ** -e < 2.0 ** 126:
            top = np.abs(capi.decode_array(fmt, codes[32 * b: 32 * b + 32][np.isfinite(blk)])).max()
            assert 2.0 ** EMAX[fmt] <= top <= 2.0 ** (EMAX[fmt] + 1)
