"""Pins for the deterministic modes of Section II-A (ties away, ties to even, ties to odd) and for the
16-bit-sum update of Algorithm 1."""
import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import FMTS, TORCH_DTYPE, bits_f32, random_f32, edge_values_f32, neighbours


@pytest.mark.parametrize("fmt", FMTS)
def test_ties_to_even_equals_torch_cast(fmt):
    """R_TNE with the exponent clamp of Eq. (2) is IEEE round-to-nearest-even: torch's narrowing cast,
    wherever the value stays in the finite range (beyond it this library saturates)."""
    rng = np.random.default_rng(40)
    lo, hi = {"bf16": (-126, 126), "fp16": (-28, 15), "e4m3": (-12, 8), "e5m2": (-19, 15)}[fmt]
    pats = np.concatenate([random_f32(rng, 20000, lo, hi), edge_values_f32()])
    x = bits_f32(pats)
    M = float(pl.FORMATS[fmt]["M"])
    ok = np.isfinite(x) & (np.abs(x) <= M)
    x = x[ok]
    got = capi.fbsr_round(x, fmt, "rtne", 1, seed=0)
    t = torch.from_numpy(x.copy()).to(TORCH_DTYPE[fmt])
    expect = t.view(torch.int16 if got.dtype == np.uint16 else torch.uint8).numpy().view(got.dtype)
    # torch rounds values just below M + ulp/2 to M as well; above that it overflows, which |x| <= M excludes
    assert np.array_equal(got, expect)


@pytest.mark.parametrize("fmt", FMTS)
def test_tie_rules_and_agreement_of_both_oracles(fmt):
    rng = np.random.default_rng(41)
    D = 24 - pl.FORMATS[fmt]["P"]
    base = 0x3F800000
    for floor_odd in (0, 1):
        tie = np.uint32(base | (floor_odd << D) | (1 << (D - 1)))              # delta exactly 1/2
        below, above = np.uint32(tie - 1), np.uint32(tie + 1)
        lo_c = neighbours(fmt, float(bits_f32(tie)))[2]
        code = lambda u, v: capi.round_one(bits_f32(u), fmt, v, 1, 0)[0]
        assert code(tie, "rta") == lo_c + 1
        assert code(tie, "rtne") == lo_c + (1 if floor_odd else 0)
        assert code(tie, "rto") == lo_c + (0 if floor_odd else 1)
        for v in ("rta", "rtne", "rto"):
            assert code(below, v) == lo_c and code(above, v) == lo_c + 1
    lo, hi = {"bf16": (-126, 126), "fp16": (-40, 17), "e4m3": (-30, 10), "e5m2": (-40, 17)}[fmt]
    for u in np.concatenate([random_f32(rng, 300, lo, hi), edge_values_f32()]):
        for v in ("rta", "rtne", "rto"):
            c1, kind, up, delta = capi.round_one(bits_f32(u), fmt, v, 1, 0)
            c0, kind0, up0, delta0 = pl.round_f32_bits(int(u), fmt, v, 0, 1)
            assert c0 == c1 and up0 == up


def test_qat_update_composition_and_stagnation():
    """w8 <- RoundTo8(w16 + u16): equals 'add in binary32, round to the 16-bit format with torch, round to 8 bits
    with the rounding oracle'; with round-to-nearest small updates never change a weight (Section IV)."""
    rng = np.random.default_rng(42)
    n = 20000
    w8 = rng.integers(0, 256, size=n).astype(np.uint8)
    w8 = w8[(w8 & 0x7F) < 0x78]                                     # finite e4m3 codes away from the top
    wv = capi.decode_array("e4m3", w8)
    u = (wv * rng.uniform(-0.2, 0.2, wv.size)).astype(np.float32)
    u16 = torch.from_numpy(u).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    uv = capi.decode_array("bf16", u16)
    s16 = torch.from_numpy((wv + uv).astype(np.float32)).to(torch.bfloat16)
    y = s16.to(torch.float32).numpy()
    for variant, k in (("srff", 3), ("srf", 3), ("src", 3), ("rtne", 1)):
        got = capi.qat_update(w8.copy(), u16, "e4m3", "bf16", variant, k, seed=6, offset=9)
        assert np.array_equal(got, capi.fbsr_round(y, "e4m3", variant, k, seed=6, offset=9))
    tiny = (wv * 0.01).astype(np.float32)                            # far below half an e4m3 ulp
    t16 = torch.from_numpy(tiny).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(capi.qat_update(w8.copy(), t16, "e4m3", "bf16", "rtne", 1, seed=0), w8)


@pytest.mark.parametrize("fmt", FMTS)
def test_paper_literal_overflow_option(fmt):
    """With the IEEE-overflow flag, nearest-even rounding of finite values beyond M matches torch's cast
    (M below M + ulp/2, then Inf; NaN for E4M3, which has no infinity); stochastic variants treat those
    values the same way, and in-range values are unaffected by the flag."""
    M = float(pl.FORMATS[fmt]["M"])
    M32 = np.float32(M)
    ulp = M32 - np.nextafter(M32, np.float32(0)) if fmt != "bf16" else np.float32(2.0 ** 120)
    ulp = np.float32(2.0 ** (np.floor(np.log2(M)) - (pl.FORMATS[fmt]["P"] - 1)))
    xs = np.array([M, np.nextafter(M32, np.float32(np.inf)), M + 0.49 * ulp, np.nextafter(np.float32(M + 0.5 * ulp), np.float32(0)),
                   M + 0.5 * ulp, M + 0.75 * ulp, M * 1.5, -(M + 0.5 * ulp), -(M + 0.25 * ulp)], dtype=np.float32)
    xs = xs[np.isfinite(xs)]
    got = capi.fbsr_round(xs, fmt + "+ieee", "rtne", 1, seed=0)
    t = torch.from_numpy(xs.copy()).to(TORCH_DTYPE[fmt])
    expect = t.view(torch.int16 if got.dtype == np.uint16 else torch.uint8).numpy().view(got.dtype)
    if fmt == "e4m3":
        # torch's NaN code carries the sign; ours too
        assert np.array_equal(got & 0x7F, expect & 0x7F)
    else:
        assert np.array_equal(got, expect)
    for variant in ("srff", "srf", "src"):
        assert np.array_equal(capi.fbsr_round(xs, fmt + "+ieee", variant, 4, seed=3), got)
    for i, x in enumerate(xs):
        c0 = pl.round_f32_bits(int(np.float32(x).view(np.uint32)), fmt, "rtne", 0, 1, ieee_overflow=True)[0]
        assert c0 == int(got[i])
    rng = np.random.default_rng(44)
    inr = (bits_f32(random_f32(rng, 2000, -10, 6))).astype(np.float32)
    assert np.array_equal(capi.fbsr_round(inr, fmt + "+ieee", "srf", 3, seed=1), capi.fbsr_round(inr, fmt, "srf", 3, seed=1))
