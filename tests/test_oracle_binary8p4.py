"""Pins for the oracle's Binary8P4 target, the format of Section IV (IEEE WG P3109, precision 4).

In the paper's notation the format is (K, P, B; M) = (8, 4, 8; 224).  The P3109 report fixes, besides these:
one zero (pattern 0x00), one NaN (pattern 0x80), +Inf = 0x7F, -Inf = 0xFF, smallest subnormal 2^-10,
smallest normal 2^-7.  torch's float8_e4m3fnuz has the same precision, bias, zero and NaN and differs only
in the all-ones magnitude (a finite 240 there, the infinity here), so its casts pin both the value of every
other code and round-to-nearest-even below M.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import VARIANTS, random_f32, bits_f32

FMT = "b8p4"


def fnuz_table():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    return codes.view(torch.float8_e4m3fnuz).to(torch.float32).numpy().astype(np.float64)


def test_format_constants_of_the_report():
    f = pl.FORMATS[FMT]
    assert (f["K"], f["P"], f["B"], f["M"]) == (8, 4, 8, 224)
    assert pl.decode(FMT, 0x7E) == 224 and capi.decode(FMT, 0x7E) == 224.0
    assert pl.decode(FMT, 0x01) == Fraction(1, 1024) and capi.decode(FMT, 0x01) == 2.0 ** -10
    assert pl.decode(FMT, 0x08) == Fraction(1, 128) and capi.decode(FMT, 0x08) == 2.0 ** -7
    assert pl.decode(FMT, 0x40) == 1 and capi.decode(FMT, 0x40) == 1.0      # exponent field 8 = the bias
    assert pl.decode(FMT, 0x7F) == "+inf" and pl.decode(FMT, 0xFF) == "-inf"
    assert capi.decode(FMT, 0x7F) == np.inf and capi.decode(FMT, 0xFF) == -np.inf
    assert pl.decode(FMT, 0x80) == "nan" and np.isnan(capi.decode(FMT, 0x80))
    assert pl.decode(FMT, 0x00) == 0 and capi.decode(FMT, 0x00) == 0.0 and not np.signbit(capi.decode(FMT, 0x00))


def test_value_function_matches_torch_fnuz_cast():
    tab = fnuz_table()
    for code in range(256):
        if code in (0x7F, 0xFF):
            continue
        v, c = pl.decode(FMT, code), capi.decode(FMT, code)
        if code == 0x80:
            assert np.isnan(tab[code]) and v == "nan" and np.isnan(c)
        else:
            assert float(v) == tab[code] == c


def test_half_the_e4m3_value_for_every_finite_code():
    """Same precision, bias one larger: each finite magnitude is half of OCP E4M3's for the same code."""
    for code in range(0x7F):
        assert pl.decode(FMT, code) == pl.decode("e4m3", code) / 2
        assert pl.decode(FMT, 0x80 | code) == -pl.decode("e4m3", code) / 2 or code == 0


def test_nearest_even_matches_torch_fnuz_cast():
    rng = np.random.default_rng(11)
    y = bits_f32(random_f32(rng, 40000, lo_exp=-14, hi_exp=7))
    y = y[np.abs(y) <= 224.0]
    # exact ties and representable values too
    tab = fnuz_table()
    fin = tab[:0x7F]
    mid = ((fin[:-1] + fin[1:]) / 2).astype(np.float32)
    y = np.concatenate([y, mid, -mid, fin.astype(np.float32), -fin.astype(np.float32)])
    want = torch.from_numpy(y).to(torch.float8_e4m3fnuz).view(torch.uint8).numpy()
    got = capi.fbsr_round(y, FMT, "rtne", 1, seed=0, offset=0)
    assert np.array_equal(got, want)
    for i in rng.integers(0, y.size, size=400):
        yb = int(y[i:i + 1].view(np.uint32)[0])
        assert pl.round_f32_bits(yb, FMT, "rtne", 0, 1)[0] == int(want[i])


@pytest.mark.parametrize("variant", VARIANTS)
def test_representable_values_are_fixed_points(variant):
    rng = np.random.default_rng(3)
    for code in range(256):
        if code in (0x7F, 0xFF, 0x80):
            continue
        v = np.float32(capi.decode(FMT, code))
        k = int(rng.integers(1, 17))
        n = (1 << k) - 1
        got, kind, up, delta = capi.round_one(v, FMT, variant, k, n)
        assert got == code and kind == 0 and up == 0 and delta == 0.0
        assert pl.round_f32_bits(int(v.view(np.uint32)), FMT, variant, n, k)[0] == code


def test_single_zero_single_nan_and_infinities():
    nan = np.uint32(0x7FC00000).view(np.float32)
    for y in (nan, -nan):
        assert capi.round_one(y, FMT, "srf", 4, 3)[0] == 0x80
        assert pl.round_f32_bits(int(np.float32(y).view(np.uint32)), FMT, "srf", 3, 4)[0] == 0x80
    assert capi.round_one(np.float32(np.inf), FMT, "srff", 2, 3)[0] == 0x7F
    assert capi.round_one(np.float32(-np.inf), FMT, "srff", 2, 3)[0] == 0xFF
    assert capi.round_one(np.float32(0.0), FMT, "srf", 1, 1)[0] == 0x00
    assert capi.round_one(np.float32(-0.0), FMT, "srf", 1, 1)[0] == 0x00
    assert pl.round_f32_bits(0x80000000, FMT, "srf", 1, 1)[0] == 0x00
    # a negative value below the smallest subnormal: rounded down it is the zero (never 0x80, the NaN),
    # rounded up it is minus the smallest subnormal
    y = np.float32(-(2.0 ** -12))                   # delta~ = 1/4
    for variant in VARIANTS + ("rtne", "rta", "rto"):
        for n in range(16):
            code, kind, up, delta = capi.round_one(y, FMT, variant, 4, n)
            assert kind == 0 and delta == 0.25
            assert code == (0x81 if up else 0x00)
            assert pl.round_f32_bits(int(y.view(np.uint32)), FMT, variant, n, 4)[0] == code
    ups = [capi.round_one(y, FMT, "srff", 4, n)[2] for n in range(16)]
    assert sum(ups) == 4                             # delta + n/16 >= 1 for n = 12..15


def test_saturation_and_ieee_overflow():
    big = np.nextafter(np.float32(224.0), np.float32(np.inf))
    for n in (0, 255):
        assert capi.round_one(big, FMT, "src", 8, n) == (0x7E, 3, 0, 0.0)
        assert capi.round_one(-big, FMT, "src", 8, n)[0] == 0xFE
    assert capi.round_one(np.float32(1e30), FMT, "srff", 3, 7)[0] == 0x7E
    # read as IEEE nearest-even beyond M: ulp(M) = 16, the tie 232 goes to M (its last bit is 0)
    ieee = FMT + "+ieee"
    assert capi.round_one(np.float32(231.9), ieee, "srff", 3, 7)[0] == 0x7E
    assert capi.round_one(np.float32(232.0), ieee, "srff", 3, 7)[0] == 0x7E
    assert capi.round_one(np.nextafter(np.float32(232.0), np.float32(1e9)), ieee, "srff", 3, 7)[0] == 0x7F
    assert capi.round_one(np.float32(-1e30), ieee, "srff", 3, 7)[0] == 0xFF
    assert pl.round_f32_bits(0x43680000, FMT, "srf", 1, 2, ieee_overflow=True)[0] == 0x7E      # 232
    assert pl.round_f32_bits(0x43680001, FMT, "srf", 1, 2, ieee_overflow=True)[0] == 0x7F
    below = np.nextafter(np.float32(224.0), np.float32(0))
    assert {capi.round_one(below, FMT, "srff", 4, n)[0] for n in range(16)} == {0x7D, 0x7E}


@pytest.mark.parametrize("variant", VARIANTS + ("rtne", "rta", "rto"))
def test_exact_rational_and_integer_tiers_agree(variant):
    rng = np.random.default_rng(17)
    ybits = np.concatenate([random_f32(rng, 1500, lo_exp=-16, hi_exp=9),
                            np.array([0, 0x80000000, 0x3A800000, 0xBA800000, 0x3A000000, 0x39FFFFFF, 0x43600000,
                                      0x43600001, 0xC3600001, 0x3C000000, 0x3BFFFFFF, 0x00000001], dtype=np.uint32)])
    for yb in ybits:
        k = int(rng.integers(1, 17))
        n = int(rng.integers(0, 1 << k))
        y = bits_f32(np.uint32(yb))
        code, kind, up, delta = capi.round_one(y, FMT, variant, k, n)
        c0, kind0, up0, delta0 = pl.round_f32_bits(int(yb), FMT, variant, n, k)
        assert (code, up) == (c0, up0) and Fraction(delta) == delta0
        assert kind == {"finite": 0, "nan": 1, "inf": 2, "sat": 3}[kind0]


@pytest.mark.parametrize("variant", VARIANTS)
def test_same_code_as_e4m3_of_twice_the_value(variant):
    """Doubling the input shifts Binary8P4's grid onto E4M3's, subnormals included, so the codes coincide
    wherever both are finite (the zero's sign apart)."""
    rng = np.random.default_rng(23)
    y = bits_f32(random_f32(rng, 20000, lo_exp=-15, hi_exp=7))
    y = y[np.abs(y) <= 224.0]
    for k in (1, 3, 4, 8, 16):
        a = capi.fbsr_round(y, FMT, variant, k, seed=5, offset=77)
        b = capi.fbsr_round((2 * y).astype(np.float32), "e4m3", variant, k, seed=5, offset=77)
        nz = (b & 0x7F) != 0
        assert np.array_equal(a[nz], b[nz]) and np.all(a[~nz] == 0)


def test_bias_closed_forms_for_bfloat16_sources():
    """Section III-E with D = 4 (BFloat16 -> precision 4) and N = 3, the setting of Section IV: mean error over
    the 16 residues is -(2^-N - 2^-D)/2 = -1/32 for SRFF, +2^-(D+1) = +1/32 for SRF, 0 for SRC."""
    D, N = 4, 3
    want = {"srff": Fraction(-1, 32), "srf": Fraction(1, 32), "src": Fraction(0)}
    for e in (-9, -3, 0, 5):                         # a subnormal binade and three normal ones
        for variant in VARIANTS:
            total = Fraction(0)
            for r in range(1 << D):
                if e == -9:
                    y = np.float32((4 + r / 16.0) * 2.0 ** -10)      # sigma~ = 4 + r/16 in the subnormal range
                else:
                    y = np.float32((1 + (8 + r / 16.0) / 8.0 - 1) * 2.0 ** e)   # significand 8 + r/16, in units of 2^(e-3)
                for n in range(1 << N):
                    code, kind, up, delta = capi.round_one(y, FMT, variant, N, n)
                    assert kind == 0 and Fraction(delta) == Fraction(r, 16)
                    total += up - Fraction(delta)
            assert total / (1 << (D + N)) == want[variant]


def test_round_array_entry_points_accept_the_format():
    rng = np.random.default_rng(5)
    x = bits_f32(random_f32(rng, 4099, lo_exp=-14, hi_exp=9))
    codes = capi.fbsr_round(x, FMT, "srf", 3, seed=1, offset=3, scale=0.5)
    for i in rng.integers(0, x.size, size=200):
        y = np.float32(x[i] * np.float32(0.5))
        n = capi.draw(1, 3 + int(i), 3)
        assert codes[i] == capi.round_one(y, FMT, "srf", 3, n)[0]
    # accumulate and the Algorithm-1 step decode and re-encode the format
    w = rng.integers(0, 256, size=2048).astype(np.uint8)
    w[(w & 0x7F) == 0x7F] = 0x30
    w[w == 0x80] = 0x00
    u = (rng.standard_normal(2048) * 0.01).astype(np.float32)
    w2 = w.copy()
    capi.accumulate(w2, u, FMT, "src", 4, seed=2, offset=0)
    for i in rng.integers(0, 2048, size=100):
        y = np.float32(np.float32(capi.decode(FMT, int(w[i]))) + u[i])
        assert w2[i] == capi.round_one(y, FMT, "src", 4, capi.draw(2, int(i), 4))[0]
