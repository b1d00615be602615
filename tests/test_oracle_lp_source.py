"""Pins for low-precision sources (BFloat16 / binary16 values rounded to 8-bit formats), the regime of
Section III-E, Fig. 2 and Algorithm 1."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import VARIANTS, TORCH_DTYPE


def widen(codes, fmt):
    """torch's own widening cast of the stored codes."""
    t = torch.from_numpy(codes.view(np.int16).copy()).view(TORCH_DTYPE[fmt])
    return t.to(torch.float32).numpy()


@pytest.mark.parametrize("src_fmt", ["bf16", "fp16"])
@pytest.mark.parametrize("dst_fmt", ["e4m3", "e5m2"])
def test_equals_rounding_of_the_widened_value(src_fmt, dst_fmt):
    """Every 16-bit code: rounding the code equals rounding torch's widening of it."""
    codes = np.arange(1 << 16, dtype=np.uint16)
    x = widen(codes, src_fmt)
    for variant, k, scale in (("srff", 3, 1.0), ("srf", 4, 0.37), ("src", 2, 1.0), ("src", 8, 3.0)):
        got = capi.fbsr_round_lp(codes, src_fmt, dst_fmt, variant, k, seed=9, offset=4, scale=scale)
        ok = ~np.isnan(x)
        expect = capi.fbsr_round(x, dst_fmt, variant, k, seed=9, offset=4, scale=scale)
        assert np.array_equal(got[ok], expect[ok])
        # NaN sources give the NaN code with the source's sign
        assert np.all((got[~ok] & 0x7F) == 0x7F) and np.array_equal(got[~ok] >> 7, (codes[~ok] >> 15).astype(np.uint8))
    # tier 0 agrees on a sample
    rng = np.random.default_rng(2)
    for c in rng.integers(0, 1 << 16, size=300):
        v = pl.decode(src_fmt, int(c))
        if isinstance(v, str):
            continue
        ybits = pl.fraction_to_f32_bits(v, negative_zero=bool(c >> 15))
        n = int(rng.integers(0, 8))
        assert pl.round_f32_bits(ybits, dst_fmt, "src", n, 3)[0] == capi.round_one(capi.decode(src_fmt, int(c)), dst_fmt, "src", 3, n)[0]


def all_draw_mean_bias(src_codes, src_fmt, dst_fmt, variant, N, ulp):
    """Mean over the given source values and over all 2^N draws of (rounded - x) / ulp, exactly."""
    x = capi.decode_array(src_fmt, src_codes).astype(np.float64)
    total = Fraction(0)
    for n in range(1 << N):
        dpw = 32 // N
        word = sum(n << (j * N) for j in range(dpw))
        words = np.full((src_codes.size + dpw - 1) // dpw, word, dtype=np.uint32)
        y = capi.decode_array(src_fmt, src_codes)
        codes = capi.fbsr_round_bits(y, dst_fmt, variant, N, words)
        err = (capi.decode_array(dst_fmt, codes).astype(np.float64) - x) / ulp
        total += Fraction(float(err.sum()))
    return total / (1 << N) / src_codes.size


@pytest.mark.parametrize("dst_fmt,D,ulp", [("e5m2", 5, 0.25), ("e4m3", 4, 0.125)])
def test_fig2_exact_bias_for_bfloat16_inputs(dst_fmt, D, ulp):
    """All 128 BFloat16 values of [1, 2) with 3 random bits: Fig. 2 prints -0.046875 / +0.015625 / 0.000
    for the precision-3 target; the precision-4 target gives the Section III-E values at D = 4."""
    codes = np.arange(0x3F80, 0x4000, dtype=np.uint16)
    expect = {"srff": (pl.pow2(-D) - pl.pow2(-3)) / 2, "srf": pl.pow2(-(D + 1)), "src": Fraction(0)}
    for variant in VARIANTS:
        assert all_draw_mean_bias(codes, "bf16", dst_fmt, variant, 3, ulp) == expect[variant]
    if dst_fmt == "e5m2":
        assert float(expect["srff"]) == -0.046875 and float(expect["srf"]) == 0.015625


def test_fig2_experiment_with_philox_draws():
    """Fig. 2 as an experiment: each BFloat16 X of [1, 2) sampled 100 000 times, 3 random bits, E5M2 target."""
    codes = np.repeat(np.arange(0x3F80, 0x4000, dtype=np.uint16), 100_000)
    x = capi.decode_array("bf16", codes).astype(np.float64)
    for variant, expect in (("srff", -0.046875), ("srf", 0.015625), ("src", 0.0)):
        out = capi.fbsr_round_lp(codes, "bf16", "e5m2", variant, 3, seed=0)
        bias = float(((capi.decode_array("e5m2", out).astype(np.float64) - x) / 0.25).mean())
        assert abs(bias - expect) < 5e-4, (variant, bias)
