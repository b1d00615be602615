"""Pins for the three few-bit predicates (Section II-B, Eq. (8)) in both oracles.

The references used here do not come from the oracles: neighbouring
representable values are taken from torch's dtype casts, delta is the exact
position between them, and the expected behaviour is what the inequalities fix.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import (FMTS, VARIANTS, EXCESS_BITS, bits_f32, edge_values_f32, random_f32,
                     neighbours, exact_delta, finite_magnitudes)


def both(ybits, fmt, variant, k, n):
    """Round one pattern in both oracles, insist they agree, return the code."""
    c1, kind, up, delta = capi.round_one(bits_f32(np.uint32(ybits)), fmt, variant, k, n)
    c0, kind0, up0, delta0 = pl.round_f32_bits(int(ybits), fmt, variant, n, k)
    assert c0 == c1, (hex(int(ybits)), fmt, variant, k, n, hex(c0), hex(c1))
    assert up0 == up and float(delta0) == delta
    assert ("finite", "nan", "inf", "sat").index(kind0) == kind
    return c1, up


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_integer_oracle_equals_rational_oracle(fmt, variant):
    rng = np.random.default_rng(100 + 10 * FMTS.index(fmt) + VARIANTS.index(variant))
    lo = {"bf16": -126, "fp16": -40, "e4m3": -30, "e5m2": -40}[fmt]
    hi = {"bf16": 127, "fp16": 17, "e4m3": 10, "e5m2": 17}[fmt]
    pats = np.concatenate([edge_values_f32(), random_f32(rng, 400, lo, hi)])
    # subnormal binary32 inputs too
    pats = np.concatenate([pats, rng.integers(1, 1 << 23, size=20, dtype=np.uint32)])
    for u in pats:
        for k in (1, 2, 3, 5, 8, 13, 16):
            for n in {0, (1 << k) - 1, int(rng.integers(0, 1 << k))}:
                both(u, fmt, variant, k, n)


@pytest.mark.parametrize("fmt", FMTS)
def test_result_is_always_a_neighbour(fmt):
    """Eq. (5): the output is floor or floor+1, i.e. one of the two representable neighbours."""
    rng = np.random.default_rng(5)
    hi = {"bf16": 100, "fp16": 14, "e4m3": 7, "e5m2": 14}[fmt]
    for u in random_f32(rng, 300, -30, hi):
        mag = abs(float(bits_f32(u)))
        lo_v, hi_v, lo_c, hi_c = neighbours(fmt, mag)
        for variant in VARIANTS:
            k = int(rng.integers(1, 17))
            n = int(rng.integers(0, 1 << k))
            code, up = both(u, fmt, variant, k, n)
            mcode = code & ((1 << (pl.FORMATS[fmt]["K"] - 1)) - 1)
            assert mcode == (hi_c if up else lo_c)
            assert (code >> (pl.FORMATS[fmt]["K"] - 1)) == int(u >> 31)


def test_srff_with_zero_draw_is_truncation_bf16():
    """n = 0 never rounds up (delta < 1), so SRFF degenerates to round-toward-zero: for
    bfloat16 that is the textbook 'keep the upper 16 bits'."""
    rng = np.random.default_rng(6)
    pats = random_f32(rng, 2000, -126, 126)
    x = bits_f32(pats)
    for k in (1, 2, 7, 16):
        words = np.zeros(pats.size, dtype=np.uint32)          # every draw is 0
        got = capi.fbsr_round_bits(x, "bf16", "srff", k, words)
        assert np.array_equal(got, (pats >> 16).astype(np.uint16))


@pytest.mark.parametrize("fmt", FMTS)
def test_extreme_draws_give_directed_rounding(fmt):
    """With N >= the number of excess bits, SRFF is exact SR: n = 0 rounds toward zero and
    n = 2^N - 1 rounds any inexact value away from zero (delta >= 2^-N)."""
    rng = np.random.default_rng(8)
    D = EXCESS_BITS[fmt]
    if D > 16:
        # restrict the inputs to 16 excess bits so that N = 16 covers them
        keep = np.uint32(0xFFFFFFFF) << np.uint32(D - 16)
    else:
        keep = np.uint32(0xFFFFFFFF)
    hi = {"bf16": 100, "fp16": 14, "e4m3": 7, "e5m2": 14}[fmt]
    lo = {"bf16": -100, "fp16": -13, "e4m3": -5, "e5m2": -13}[fmt]     # normal range of the target
    for u in random_f32(rng, 500, lo, hi) & keep:
        mag = abs(float(bits_f32(u)))
        _, _, lo_c, hi_c = neighbours(fmt, mag)
        mask = (1 << (pl.FORMATS[fmt]["K"] - 1)) - 1
        for variant in VARIANTS:
            assert both(u, fmt, variant, 16, 0)[0] & mask == lo_c
            assert both(u, fmt, variant, 16, 0xFFFF)[0] & mask == hi_c


def expected_up_count(variant, delta, N):
    """Number of draws n in [0, 2^N) for which the printed inequality holds."""
    z = delta * (1 << N)
    if variant == "srff":      # delta + n 2^-N >= 1  <=>  n >= 2^N - z  -> floor(z) draws
        return z.numerator // z.denominator
    if variant == "srf":       # n >= 2^N - z - 1/2  -> floor(z + 1/2) draws
        zz = z + Fraction(1, 2)
        return zz.numerator // zz.denominator
    fl = z.numerator // z.denominator
    d = z - fl
    if d > Fraction(1, 2) or (d == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl                  # SRC: nearest-even of z draws


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_exhaustive_draws_give_the_exact_round_up_probability(fmt, variant):
    """Counting round-ups over all 2^N draws: floor, round-half-up and round-half-even of
    delta 2^N for SRFF, SRF and SRC.  delta comes from the neighbour table, not the oracle."""
    rng = np.random.default_rng(200 + 10 * FMTS.index(fmt) + VARIANTS.index(variant))
    hi = {"bf16": 100, "fp16": 14, "e4m3": 7, "e5m2": 14}[fmt]
    lo = {"bf16": -126, "fp16": -26, "e4m3": -11, "e5m2": -18}[fmt]    # includes target subnormals
    pats = list(random_f32(rng, 60, lo, hi))
    # values with few excess bits and exact ties for the SRC pre-round
    base = {"bf16": 0x3F800000, "fp16": 0x3F800000, "e4m3": 0x3F800000, "e5m2": 0x3F800000}[fmt]
    D = EXCESS_BITS[fmt]
    for frac in (1, 2, 3, 5, 6, 7, 8, 10, 12, 14, 15):
        pats.append(np.uint32(base | (frac << (D - 4))))           # delta = frac/16
        pats.append(np.uint32(base | (1 << D) | (frac << (D - 4))))  # odd floor
    for u in pats:
        mag = abs(float(bits_f32(np.uint32(u))))
        delta = exact_delta(fmt, mag)
        for N in (1, 2, 3, 4, 6):
            ups = sum(capi.round_one(bits_f32(np.uint32(u)), fmt, variant, N, n)[2] for n in range(1 << N))
            assert ups == expected_up_count(variant, delta, N), (hex(int(u)), N, delta)
        # tier 0 on a subset
        ups0 = sum(pl.round_f32_bits(int(u), fmt, variant, n, 3)[2] for n in range(8))
        assert ups0 == expected_up_count(variant, delta, 3)


@pytest.mark.parametrize("fmt,N", [("bf16", 16), ("fp16", 13), ("fp16", 16)])
@pytest.mark.parametrize("variant", VARIANTS)
def test_enough_bits_is_exact_stochastic_rounding(fmt, N, variant):
    """N >= excess bits: the mean over all draws reproduces the input exactly (P_up = delta)."""
    rng = np.random.default_rng(9)
    lo, hi = {"bf16": (-120, 120), "fp16": (-13, 15)}[fmt]
    for u in random_f32(rng, 6, lo, hi):
        x = bits_f32(u)
        xs = np.full(1 << N, x, dtype=np.float32)
        words = np.arange(1 << N, dtype=np.uint32) if 32 // N == 1 else None
        if words is None:
            dpw = 32 // N
            n_all = np.arange(1 << N, dtype=np.uint64)
            words = np.zeros((1 << N) // dpw + 1, dtype=np.uint32)
            for j in range(dpw):
                sel = n_all[j::dpw]
                words[:sel.size] |= (sel << np.uint64(j * N)).astype(np.uint32)
        codes = capi.fbsr_round_bits(xs, fmt, variant, N, words)
        vals = capi.decode_array(fmt, codes).astype(np.float64)
        assert Fraction(float(vals.sum())) / (1 << N) == Fraction(float(x))


def test_src_to_e5m2_with_8_bits_is_half_precision_rtne_then_srff():
    """Eq. (8) with P = 3, N = 8 pre-rounds to precision 11 on E5M2's exponent range, which
    is IEEE binary16.  So SRC(x) must equal SRFF applied to torch's round-to-nearest-even
    half-precision cast of x."""
    rng = np.random.default_rng(10)
    pats = np.concatenate([random_f32(rng, 4000, -27, 15), edge_values_f32()])
    x = bits_f32(pats)
    ok = np.isfinite(x) & (np.abs(x) <= 57344.0)
    x = x[ok]
    words = rng.integers(0, 1 << 32, size=x.size, dtype=np.uint32)   # 4 fields of 8 bits per word
    src = capi.fbsr_round_bits(x, "e5m2", "src", 8, words)
    xh = torch.from_numpy(x.copy()).to(torch.float16).to(torch.float32).numpy()
    srff = capi.fbsr_round_bits(xh, "e5m2", "srff", 8, words)
    assert np.array_equal(src, srff)


def test_sign_symmetry():
    rng = np.random.default_rng(12)
    pats = random_f32(rng, 500, -20, 10)
    for fmt in FMTS:
        top = 1 << (pl.FORMATS[fmt]["K"] - 1)
        for variant in VARIANTS:
            k = 4
            for u in pats[:100]:
                n = int(rng.integers(0, 16))
                a = capi.round_one(bits_f32(u), fmt, variant, k, n)[0]
                b = capi.round_one(bits_f32(u ^ np.uint32(0x80000000)), fmt, variant, k, n)[0]
                assert a ^ b == top


def test_scale_is_one_rounded_multiply():
    rng = np.random.default_rng(13)
    x = bits_f32(random_f32(rng, 2000, -10, 10))
    scale = np.float32(3.1415927)
    y = (x * scale).astype(np.float32)           # numpy's binary32 multiply, one rounding
    for fmt in ("e4m3", "fp16"):
        a = capi.fbsr_round(x, fmt, "srf", 4, seed=5, offset=3, scale=float(scale))
        b = capi.fbsr_round(y, fmt, "srf", 4, seed=5, offset=3, scale=1.0)
        assert np.array_equal(a, b)
    # tier 0 uses an exact product rounded once: same thing
    sb = int(scale.view(np.uint32))
    codes0, _ = pl.fbsr_round([int(v) for v in x[:200].view(np.uint32)], "e4m3", "srf", 4, 5, 3, sb)
    assert codes0 == list(capi.fbsr_round(x[:200], "e4m3", "srf", 4, 5, 3, float(scale)))


def test_array_call_is_elementwise_with_global_index():
    """Shards with offsets reproduce the single call; Philox path == supplied-words path."""
    rng = np.random.default_rng(14)
    x = bits_f32(random_f32(rng, 1000, -10, 10))
    for k in (2, 3, 6, 13):
        whole = capi.fbsr_round(x, "fp16", "srf", k, seed=77, offset=0)
        parts = [capi.fbsr_round(x[a:b], "fp16", "srf", k, seed=77, offset=a)
                 for a, b in ((0, 333), (333, 334), (334, 1000))]
        assert np.array_equal(whole, np.concatenate(parts))
        words = capi.random_words(77, 0, x.size, k)
        assert np.array_equal(whole, capi.fbsr_round_bits(x, "fp16", "srf", k, words))
        one_by_one = [capi.round_one(x[i], "fp16", "srf", k, capi.draw(77, i, k))[0] for i in range(50)]
        assert list(whole[:50]) == one_by_one


@pytest.mark.parametrize("fmt", FMTS + ("b8p4",))
@pytest.mark.parametrize("variant", VARIANTS + ("rtne", "rta", "rto"))
def test_rounding_is_monotone_in_the_magnitude(fmt, variant):
    """For a fixed draw, floor(sigma~) + [R] never decreases when the value grows (each predicate is monotone in
    delta~, and a larger floor outweighs any predicate), and codes of positive values are ordered like the values:
    sorted magnitudes must give non-decreasing codes, through binade changes, the subnormal range and saturation."""
    rng = np.random.default_rng(97)
    lo, hi = {"bf16": (-126, 127), "fp16": (-30, 17), "e4m3": (-14, 10), "e5m2": (-22, 17), "b8p4": (-15, 9)}[fmt]
    mags = np.sort(bits_f32(random_f32(rng, 30000, lo, hi) & np.uint32(0x7FFFFFFF)))
    # and a dense run of consecutive binary32 values across a rounding boundary
    mags = np.concatenate([mags, bits_f32(np.arange(0x3F7FFF00, 0x3F800100, dtype=np.uint32))])
    mags = np.sort(mags)
    for k in (1, 3, 7, 16):
        for n in (0, (1 << k) // 3, (1 << k) - 1):
            words_n = n
            codes = np.array([capi.round_one(y, fmt, variant, k, words_n)[0] for y in mags[::7]], dtype=np.int64)
            assert np.all(np.diff(codes) >= 0), (fmt, variant, k, n)
