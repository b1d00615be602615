"""Pins for Eq. (1) (value of a code) and for encoding: torch's dtype casts are the reference."""
import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import FMTS, VARIANTS, CODE_BITS, TORCH_DTYPE, torch_decode_table, finite_magnitudes


@pytest.mark.parametrize("fmt", FMTS)
def test_value_function_matches_torch_cast(fmt):
    """Every code, widened by Eq. (1), equals torch's widening cast of the same bits."""
    tab = torch_decode_table(fmt)
    for code in range(1 << CODE_BITS[fmt]):
        v = pl.decode(fmt, code)
        c = capi.decode(fmt, code)
        if v == "nan":
            assert np.isnan(tab[code]) and np.isnan(c)
        elif v in ("+inf", "-inf"):
            assert np.isinf(tab[code]) and (tab[code] > 0) == (v == "+inf") and c == tab[code]
        else:
            assert float(v) == tab[code] and c == tab[code]
            assert np.signbit(c) == bool(code >> (CODE_BITS[fmt] - 1))


@pytest.mark.parametrize("fmt", FMTS)
def test_largest_finite_value(fmt):
    f = pl.FORMATS[fmt]
    vals, codes = finite_magnitudes(fmt)
    assert float(f["M"]) == vals[-1] and f["max_code"] == codes[-1]
    assert pl.decode(fmt, f["max_code"]) == f["M"]
    # torch's own finfo agrees on M
    assert float(torch.finfo(TORCH_DTYPE[fmt]).max) == float(f["M"])


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_representable_values_are_fixed_points(fmt, variant):
    """delta = 0 can never satisfy a predicate (delta + anything < 1): exact inputs map to themselves."""
    tab = torch_decode_table(fmt)
    rng = np.random.default_rng(3)
    for code in range(1 << CODE_BITS[fmt]):
        v = tab[code]
        if not np.isfinite(v):
            continue
        k = int(rng.integers(1, 17))
        n = (1 << k) - 1                      # the draw most likely to round up
        got, kind, up, delta = capi.round_one(np.float32(v), fmt, variant, k, n)
        assert got == code and kind == 0 and up == 0 and delta == 0.0
        ybits = int(np.float32(v).view(np.uint32))
        assert pl.round_f32_bits(ybits, fmt, variant, n, k)[0] == code


@pytest.mark.parametrize("fmt", FMTS)
def test_specials_and_saturation_policy(fmt):
    f = pl.FORMATS[fmt]
    top = 1 << (f["K"] - 1)
    nan = np.uint32(0x7FC00000).view(np.float32)
    assert capi.round_one(nan, fmt, "srf", 4, 3)[0] == f["nan_code"]
    assert capi.round_one(-nan, fmt, "srf", 4, 3)[0] == top | f["nan_code"]
    inf_code = f["inf_code"] if f["inf_code"] is not None else f["max_code"]
    assert capi.round_one(np.float32(np.inf), fmt, "srff", 2, 3)[0] == inf_code
    assert capi.round_one(np.float32(-np.inf), fmt, "srff", 2, 3)[0] == top | inf_code
    big = np.nextafter(np.float32(float(f["M"])), np.float32(np.inf))
    for n in (0, 255):
        code, kind, up, _ = capi.round_one(big, fmt, "src", 8, n)
        assert code == f["max_code"] and kind == 3 and up == 0
        assert capi.round_one(-big, fmt, "src", 8, n)[0] == top | f["max_code"]
    # just below M rounds to M or its predecessor, never beyond
    below = np.nextafter(np.float32(float(f["M"])), np.float32(0))
    for n in range(16):
        code = capi.round_one(below, fmt, "srff", 4, n)[0]
        assert code in (f["max_code"], f["max_code"] - 1)
    assert capi.round_one(np.float32(0.0), fmt, "srf", 1, 1)[0] == 0
    assert capi.round_one(np.float32(-0.0), fmt, "srf", 1, 1)[0] == top
