"""Small helpers shared by the test modules (no method arithmetic)."""
import os
from fractions import Fraction

import numpy as np
import torch

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
FMTS = ("bf16", "fp16", "e4m3", "e5m2")       # the formats torch has a dtype for
ALL_FMTS = FMTS + ("b8p4",)                    # plus Section IV's Binary8P4
VARIANTS = ("srff", "srf", "src")
TORCH_DTYPE = {"bf16": torch.bfloat16, "fp16": torch.float16,
               "e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}
CODE_BITS = {"bf16": 16, "fp16": 16, "e4m3": 8, "e5m2": 8}
EXCESS_BITS = {"bf16": 16, "fp16": 13, "e4m3": 20, "e5m2": 21}   # 24 - P


def f32_bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def bits_f32(u):
    return np.asarray(u, dtype=np.uint32).view(np.float32)


def torch_decode_table(fmt):
    """Every code of the format widened to float64 by torch's own dtype cast."""
    nbits = CODE_BITS[fmt]
    codes = torch.arange(1 << nbits, dtype=torch.int32)
    raw = codes.to(torch.uint8) if nbits == 8 else codes.to(torch.int16)
    return raw.view(TORCH_DTYPE[fmt]).to(torch.float32).numpy().astype(np.float64)


def finite_magnitudes(fmt):
    """Sorted array of the non-negative finite values of the format (float64), with their codes."""
    tab = torch_decode_table(fmt)
    half = 1 << (CODE_BITS[fmt] - 1)
    vals = tab[:half]
    ok = np.isfinite(vals)
    codes = np.nonzero(ok)[0]
    return vals[ok], codes      # already ascending: encodings of positive values are monotone


def neighbours(fmt, mag):
    """(lo_value, hi_value, lo_code, hi_code) bracketing the magnitude, lo <= mag <= hi."""
    vals, codes = finite_magnitudes(fmt)
    i = int(np.searchsorted(vals, mag, side="right")) - 1
    if vals[i] == mag:
        return vals[i], vals[i], int(codes[i]), int(codes[i])
    return vals[i], vals[i + 1], int(codes[i]), int(codes[i + 1])


def exact_delta(fmt, mag):
    """Fractional position of mag between its two neighbours, as a Fraction."""
    lo, hi, _, _ = neighbours(fmt, mag)
    if lo == hi:
        return Fraction(0)
    return (Fraction(float(mag)) - Fraction(lo)) / (Fraction(hi) - Fraction(lo))


def edge_values_f32():
    """Binary32 patterns that exercise every special path."""
    u = [0x00000000, 0x80000000, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0xFF7FFFFF,
         0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00001, 0x7F800001, 0x3F800000, 0xBF800000,
         0x3F7FFFFF, 0x3F808000, 0x3F818000, 0x3F80FFFF, 0x7F7F0000, 0x7F7F0001, 0x7F7E8000,
         0x477FE000, 0x477FE001, 0x477FF000, 0x47800000, 0x43E00000, 0x43E00001, 0x43E80000,
         0x43F00000, 0x47600000, 0x47600001, 0x47700000, 0x33800000, 0x33000000, 0x32FFFFFF,
         0x38800000, 0x387FFFFF, 0x38000000, 0x3C800000, 0x3C7FFFFF, 0x3B000000, 0x3A800000,
         0x3A7FFFFF, 0x37800000, 0x37000000, 0x36FFFFFF, 0x1E000000, 0x0D000000]
    return np.array(u, dtype=np.uint32)


def random_f32(rng, n, lo_exp=-30, hi_exp=20):
    """Random finite binary32 values with log-uniform magnitude and random sign."""
    mant = rng.integers(0, 1 << 23, size=n, dtype=np.uint32)
    exp = rng.integers(lo_exp + 127, hi_exp + 127 + 1, size=n, dtype=np.uint32)
    sign = rng.integers(0, 2, size=n, dtype=np.uint32)
    return ((sign << np.uint32(31)) | (exp << np.uint32(23)) | mant).astype(np.uint32)
