"""The oracle reproduces the bias values and closed forms the paper states (Section III,
Appendices A-D, captions of Fig. 1 and Fig. 2)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import capi, paper_literal as pl
from helpers import GOLDEN, VARIANTS, bits_f32


def constant_draw_words(count, k, n):
    dpw = 32 // k
    pat = 0
    for j in range(dpw):
        pat |= n << (j * k)
    return np.full((count + dpw - 1) // dpw, pat, dtype=np.uint32)


def mean_bias_over_residues(fmt, variant, N, D, base_bits, excess):
    """Exact mean over all 2^D residues and all 2^N draws of (rounded - x) in target ulps.

    base_bits: a binary32 pattern whose low `excess` bits are zero (an exact target value);
    the residues fill the top D of those bits.  The error is measured from the decoded
    outputs, not from the oracle's own delta."""
    i = np.arange(1 << D, dtype=np.uint32)
    pats = np.uint32(base_bits) | (i << np.uint32(excess - D))
    x = bits_f32(pats)
    ulp = float(bits_f32(np.uint32(base_bits + (1 << excess)))) - float(bits_f32(np.uint32(base_bits)))
    total = Fraction(0)
    for n in range(1 << N):
        codes = capi.fbsr_round_bits(x, fmt, variant, N, constant_draw_words(x.size, N, n))
        vals = capi.decode_array(fmt, codes).astype(np.float64)
        err = (vals - x.astype(np.float64)) / ulp          # exact: dyadic, few bits
        total += Fraction(float(err.sum()))
    return total / (1 << N) / (1 << D)


def paper_rows():
    rows = []
    with open(os.path.join(GOLDEN, "paper_bias_values.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                t = line.split()
                rows.append((t[0], int(t[1]), t[2], float(t[3])))
    return rows


@pytest.mark.parametrize("variant,N,D,value", paper_rows())
def test_values_printed_in_the_paper(variant, N, D, value):
    if D == "inf":
        # continuous input: binary32 into bfloat16 leaves 16 excess bits; the finite-D closed
        # forms differ from the continuous ones by 2^-17, far below what the figure resolves.
        got = mean_bias_over_residues("bf16", variant, N, 16, 0x3F800000, 16)
        assert abs(float(got) - value) <= 2.0 ** -17
    else:
        # Fig. 2: BFloat16-precision inputs (8 bits) into a precision-3 target: D = 5.
        D = int(D)
        got = mean_bias_over_residues("e5m2", variant, N, D, 0x3F800000, 21)
        assert float(got) == value


@pytest.mark.parametrize("N,D", [(1, 3), (2, 3), (2, 4), (2, 5), (3, 5), (4, 8), (1, 16), (2, 16),
                                 (4, 16), (8, 16), (4, 4), (8, 8), (13, 13), (10, 8), (6, 3)])
def test_closed_forms_for_finite_precision_inputs(N, D):
    """Section III-E: SRFF (2^-D - 2^-N)/2 for N <= D; SRF 2^-(D+1) for N < D; SRC 0;
    everything 0 once N >= D.  Inputs: binary32 values with exactly D bits below a
    bfloat16 (D <= 16) or binary16 (D <= 13) lsb."""
    fmt, excess = ("fp16", 13) if D <= 13 and (N + D) % 2 else ("bf16", 16)
    base = 0x3F800000 | (3 << excess)
    srff = mean_bias_over_residues(fmt, "srff", N, D, base, excess)
    srf = mean_bias_over_residues(fmt, "srf", N, D, base, excess)
    src = mean_bias_over_residues(fmt, "src", N, D, base, excess)
    if N <= D:
        assert srff == (pl.pow2(-D) - pl.pow2(-N)) / 2
    else:
        assert srff == 0
    assert srf == (pl.pow2(-(D + 1)) if N < D else 0)
    assert src == 0
    # the unsimplified sums of Appendices C and D agree as well
    assert srff == pl.bias_srff_finite(N, D)
    assert srf == pl.bias_srf_finite(N, D)


def test_bias_also_holds_in_the_subnormal_range_and_other_binades():
    """Eq. (2) gives subnormals a fixed lsb, so the same closed forms hold there."""
    # binary16 subnormal range: lsb 2^-24; take values 2^-20 * (1 + ...) -> excess bits 13 + 6
    # use D = 4 residues directly below the subnormal lsb.
    base = int(np.float32(2.0 ** -20).view(np.uint32))       # exact binary16 subnormal
    # in binary32 this value has exponent -20, lsb 2^-43; target lsb 2^-24 -> 19 excess bits
    got = mean_bias_over_residues("fp16", "srff", 2, 4, base, 19)
    assert got == (pl.pow2(-4) - pl.pow2(-2)) / 2
    assert mean_bias_over_residues("fp16", "srf", 2, 4, base, 19) == pl.pow2(-5)
    assert mean_bias_over_residues("fp16", "src", 2, 4, base, 19) == 0
    # a different binade of E4M3 with an odd significand
    base = int(np.float32(13.0).view(np.uint32))
    assert mean_bias_over_residues("e4m3", "srff", 3, 6, base, 20) == (pl.pow2(-6) - pl.pow2(-3)) / 2


def bias_grid(primary):
    i = np.arange(1024, dtype=np.float64)
    X = 1.0 + ((2 * i + 1) / 2048.0 if primary else i / 1024.0)
    return np.repeat(X.astype(np.float32), 5000)


@pytest.mark.parametrize("primary,expect", [(True, {"srff": -0.125, "srf": 0.0, "src": 0.0}),
                                            (False, {"srff": -0.0625, "srf": 0.0625, "src": 0.0})])
def test_fig1_experiment_with_philox_draws(primary, expect):
    """Fig. 1 set-up: 1024 X values across [1, 2), 5000 samples each, 2 random bits, bfloat16.
    Cell-centred X (4 excess bits, odd residues) gives the continuous-input biases
    -2^-3 / 0 / 0; X on the 1/1024 grid has 3 excess bits, so Section III-E predicts
    -2^-4 / +2^-4 / 0.  Sampling error of the overall mean is about 2e-4 ulp."""
    x = bias_grid(primary)
    for variant in VARIANTS:
        codes, st, ge, ge2 = capi.fbsr_round_stats(x, "bf16", variant, 2, seed=0, group_size=5000)
        assert st["n_finite"] == x.size and st["n_nan"] == st["n_inf"] == st["n_sat"] == 0
        bias = st["sum_e"] / st["n_finite"]
        assert abs(bias - expect[variant]) < 1e-3, (variant, bias)
        # the same number measured from the decoded outputs
        vals = capi.decode_array("bf16", codes).astype(np.float64)
        bias2 = float(((vals - x.astype(np.float64)) * 128.0).mean())
        assert abs(bias - bias2) < 1e-12
        assert abs(ge.sum() - st["sum_e"]) < 1e-6
        # per-X means: within 5 standard errors of the exact per-value expectation
        per_x = ge / 5000.0
        frac16 = (x[::5000].view(np.uint32) & 0xFFFF).astype(np.float64) / 65536.0   # delta
        z = frac16 * 4
        p_up = {"srff": np.floor(z), "srf": np.floor(z + 0.5),
                "src": np.floor(z + 0.5) - ((z % 1 == 0.5) & (np.floor(z + 0.5) % 2 == 1))}[variant] / 4
        assert np.all(np.abs(per_x - (p_up - frac16)) < 5 * 0.5 / np.sqrt(5000.0) + 1e-12)


def test_stats_definition_against_exact_sums():
    """sum_e, sum_e2, ... from the C oracle equal the exact rational sums of up - delta."""
    rng = np.random.default_rng(21)
    from helpers import random_f32, edge_values_f32
    pats = np.concatenate([random_f32(rng, 300, -30, 18), edge_values_f32()])
    x = bits_f32(pats)
    for fmt, k in (("fp16", 3), ("e4m3", 4), ("bf16", 2)):
        codes, st, ge, ge2 = capi.fbsr_round_stats(x, fmt, "srf", k, seed=4, offset=5, scale=1.5, group_size=7)
        sb = int(np.float32(1.5).view(np.uint32))
        codes0, st0 = pl.fbsr_round([int(v) for v in pats], fmt, "srf", k, 4, 5, sb)
        assert list(codes) == codes0
        for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
            assert st[key] == st0[key]
        for key in ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e"):
            assert abs(st[key] - float(st0[key])) <= 1e-12 * max(1.0, abs(float(st0[key])))
        e = [Fraction(0) if v is None else v for v in st0["e"]]
        for g in range(len(ge)):
            assert abs(ge[g] - float(sum(e[7 * g:7 * g + 7]))) < 1e-12
            assert abs(ge2[g] - float(sum(v * v for v in e[7 * g:7 * g + 7]))) < 1e-12
