"""Pins for formats (K, P, B; M) described at run time (Section II's parametrisation).

Independent references: torch's float8_e4m3fnuz = (8, 4, 8; 240) and float8_e5m2fnuz = (8, 3, 16; 57344), both with
one zero, one NaN (0x80) and no infinity, which none of the built-in formats is; and every built-in format written
as a descriptor must reproduce the built-in results (those are pinned to torch's other dtypes elsewhere).
"""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import VARIANTS, random_f32, bits_f32

# name -> (K, P, B, max_code, inf_code, nan_code, single_zero)
BUILTIN = {
    "bf16": (16, 8, 127, 0x7F7F, 0x7F80, 0x7FC0, False),
    "fp16": (16, 11, 15, 0x7BFF, 0x7C00, 0x7E00, False),
    "e4m3": (8, 4, 7, 0x7E, None, 0x7F, False),
    "e5m2": (8, 3, 15, 0x7B, 0x7C, 0x7F, False),
    "b8p4": (8, 4, 8, 0x7E, 0x7F, 0x80, True),
}
FNUZ = {
    "e4m3fnuz": ((8, 4, 8, 0x7F, None, 0x80, True), torch.float8_e4m3fnuz, 240.0),
    "e5m2fnuz": ((8, 3, 16, 0x7F, None, 0x80, True), torch.float8_e5m2fnuz, 57344.0),
}
RANGE = {"bf16": (-126, 127), "fp16": (-28, 17), "e4m3": (-13, 10), "e5m2": (-20, 17), "b8p4": (-14, 9)}


@pytest.mark.parametrize("name", sorted(FNUZ))
def test_value_of_every_code_matches_torch_fnuz(name):
    args, dtype, M = FNUZ[name]
    d, f = capi.make_desc(*args), pl.make_format(*args)
    assert capi.desc_valid(d) and f["M"] == M
    tab = torch.arange(256, dtype=torch.int32).to(torch.uint8).view(dtype).to(torch.float32).numpy()
    for code in range(256):
        v, c = pl.decode(f, code), capi.decode_desc(d, code)
        if code == 0x80:
            assert v == "nan" and np.isnan(c) and np.isnan(tab[code])
        else:
            assert float(v) == float(tab[code]) == c


@pytest.mark.parametrize("name", sorted(FNUZ))
def test_nearest_even_matches_torch_fnuz_cast(name):
    args, dtype, M = FNUZ[name]
    d, f = capi.make_desc(*args), pl.make_format(*args)
    rng = np.random.default_rng(31)
    hi = int(np.log2(M))
    y = bits_f32(random_f32(rng, 30000, lo_exp=hi - 24, hi_exp=hi))
    y = y[np.abs(y) <= M]
    tab = torch.arange(128, dtype=torch.int32).to(torch.uint8).view(dtype).to(torch.float32).numpy()
    mid = ((tab[:-1].astype(np.float64) + tab[1:]) / 2).astype(np.float32)       # exact ties
    y = np.concatenate([y, mid, -mid, tab, -tab])
    want = torch.from_numpy(y).to(dtype).view(torch.uint8).numpy()
    got = capi.fbsr_round_desc(y, d, "rtne", 1, seed=0)
    assert np.array_equal(got, want)
    for i in rng.integers(0, y.size, size=300):
        assert pl.round_f32_bits(int(y[i:i + 1].view(np.uint32)[0]), f, "rtne", 0, 1)[0] == int(want[i])
    # no infinity: an infinite input saturates; with the IEEE reading of overflow it becomes the NaN
    assert capi.round_one_desc(np.float32(np.inf), d, "srf", 2, 1)[0] == 0x7F
    assert capi.round_one_desc(np.float32(-np.inf), d, "srf", 2, 1)[0] == 0xFF
    assert capi.round_one_desc(np.float32(1e30), d, "srf", 2, 1, ieee_overflow=True)[0] == 0x80
    assert pl.round_f32_bits(0x7149F2CA, f, "srf", 1, 2, ieee_overflow=True)[0] == 0x80


@pytest.mark.parametrize("name", sorted(BUILTIN))
def test_builtin_formats_as_descriptors(name):
    d, f = capi.make_desc(*BUILTIN[name]), pl.make_format(*BUILTIN[name])
    assert capi.desc_valid(d) and f["M"] == pl.FORMATS[name]["M"]
    K = BUILTIN[name][0]
    rng = np.random.default_rng(37)
    for code in rng.integers(0, 1 << K, size=2000):
        a, b = capi.decode_desc(d, int(code)), capi.decode(name, int(code))
        assert (np.isnan(a) and np.isnan(b)) or (a == b and np.signbit(a) == np.signbit(b))
        assert pl.decode(f, int(code)) == pl.decode(name, int(code))
    lo, hi = RANGE[name]
    x = bits_f32(np.concatenate([random_f32(rng, 6000, lo, hi),
                                 np.array([0, 0x80000000, 0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00000, 1, 0x80000001],
                                          dtype=np.uint32)]))
    for variant in VARIANTS + ("rtne", "rta", "rto"):
        for k in (1, 3, 8, 16):
            for ieee in (False, True):
                want = capi.fbsr_round(x, name + ("+ieee" if ieee else ""), variant, k, seed=4, offset=9, scale=1.5)
                got = capi.fbsr_round_desc(x, d, variant, k, seed=4, offset=9, scale=1.5, ieee_overflow=ieee)
                assert np.array_equal(got, want)
    for i in rng.integers(0, x.size, size=200):
        yb = int(x[i:i + 1].view(np.uint32)[0])
        n = int(rng.integers(0, 8))
        assert pl.round_f32_bits(yb, f, "src", n, 3) == pl.round_f32_bits(yb, name, "src", n, 3)


def test_exact_rational_and_integer_tiers_agree_on_odd_formats():
    """Formats that no library has: (8, 2, 32), (8, 6, 2), (16, 13, 4), (16, 5, 127) with assorted tops."""
    rng = np.random.default_rng(41)
    for args in ((8, 2, 32, 0x7D, 0x7E, 0x7F, False), (8, 6, 2, 0x5F, None, 0x7F, False),
                 (16, 13, 4, 0x7FFE, None, 0x8000, True), (16, 5, 127, 0x0FEF, 0x0FF0, 0x0FF8, False)):
        d, f = capi.make_desc(*args), pl.make_format(*args)
        assert capi.desc_valid(d)
        P, B = args[1], args[2]
        hi = min(int(np.floor(np.log2(float(f["M"])))) + 2, 127)
        lo = max(2 - B - P - 3, -140)
        ybits = random_f32(rng, 600, lo_exp=max(lo, -126), hi_exp=hi)
        ybits = np.concatenate([ybits, rng.integers(0, 1 << 23, size=40, dtype=np.uint32)])       # binary32 subnormals
        for yb in ybits:
            for variant in VARIANTS + ("rtne",):
                k = int(rng.integers(1, 17))
                n = int(rng.integers(0, 1 << k))
                for ieee in (False, True):
                    code, kind, up, delta = capi.round_one_desc(bits_f32(np.uint32(yb)), d, variant, k, n, ieee_overflow=ieee)
                    c0, kind0, up0, delta0 = pl.round_f32_bits(int(yb), f, variant, n, k, ieee_overflow=ieee)
                    assert (code, up) == (c0, up0) and Fraction(delta) == delta0
        # representable values are fixed points
        for code in rng.integers(0, args[3] + 1, size=200):
            v = np.float32(capi.decode_desc(d, int(code)))
            assert capi.round_one_desc(v, d, "srf", 5, 31)[0] == int(code)


def test_bias_closed_forms_on_a_custom_precision():
    """Section III-E for a precision-6 target fed BFloat16-precision values: D = 2 excess bits.  With N = 1:
    SRFF -(2^-1 - 2^-2)/2 = -1/8, SRF +2^-3, SRC 0; with N >= D every variant is exact SR (bias 0)."""
    d = capi.make_desc(8, 6, 2, 0x5F, None, 0x7F, False)
    for N, want in ((1, {"srff": Fraction(-1, 8), "srf": Fraction(1, 8), "src": Fraction(0)}),
                    (2, {"srff": Fraction(0), "srf": Fraction(0), "src": Fraction(0)}),
                    (5, {"srff": Fraction(0), "srf": Fraction(0), "src": Fraction(0)})):
        for variant in VARIANTS:
            total = Fraction(0)
            for r in range(4):
                y = np.float32((32 + r / 4.0) / 32.0)            # significand 32 + r/4 in units of 2^-5
                for n in range(1 << N):
                    code, kind, up, delta = capi.round_one_desc(y, d, variant, N, n)
                    assert kind == 0 and Fraction(delta) == Fraction(r, 4)
                    total += up - Fraction(delta)
            assert total / (4 << N) == want[variant], (N, variant)


def test_rejected_descriptors():
    ok = (8, 4, 7, 0x7E, None, 0x7F, False)
    assert capi.desc_valid(capi.make_desc(*ok))
    for bad in ((12, 4, 7, 0x7E, None, 0x7F, False),        # K
                (8, 1, 7, 0x7E, None, 0x7F, False),         # P too small
                (8, 8, 7, 0x7E, None, 0x7F, False),         # no exponent field left
                (16, 14, 7, 0x7E, None, 0x7FFF, False),     # P beyond 13
                (8, 4, 0, 0x7E, None, 0x7F, False),         # B
                (8, 4, 128, 0x7E, None, 0x7F, False),
                (8, 4, 7, 0x00, None, 0x7F, False),         # no finite value
                (8, 4, 7, 0x7E, 0x7E, 0x7F, False),         # infinity not above M
                (8, 4, 7, 0x7E, 0x7F, 0x7F, False),         # NaN and infinity collide
                (8, 4, 7, 0x7E, None, 0x7D, False),         # NaN not above M
                (8, 4, 7, 0x7E, None, 0x7F, True),          # single zero wants NaN = 0x80
                (16, 8, 100, 0x7F7F, 0x7F80, 0x7FC0, False)):   # M beyond binary32: exponent 254 - 100 > 127
        assert not capi.desc_valid(capi.make_desc(*bad)), bad
