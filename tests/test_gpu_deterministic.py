"""GPU parity for the deterministic modes (Section II-A) and the 16-bit-sum update of Algorithm 1."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import FMTS, TORCH_DTYPE  # noqa: E402

DET = ("rtne", "rta", "rto")


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from paper_2504_20634_b200 import workloads
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu, module.workloads = fbsr, capi, gpu_util, workloads


@pytest.mark.parametrize("fmt", FMTS)
def test_deterministic_modes_everywhere(fmt):
    """Random patterns over the whole binary32 range plus exact ties of every floor parity; tiles and ragged end;
    also through the statistics and supplied-bits entry points (which must ignore the draws)."""
    rng = np.random.default_rng(90 + FMTS.index(fmt))
    n = 9 * 1024 + 55
    pats = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    D = 24 - {"bf16": 8, "fp16": 11, "e4m3": 4, "e5m2": 3}[fmt]
    ties = (np.uint32(0x3F800000) + (rng.integers(0, 1 << (23 - D), size=2000).astype(np.uint32) << np.uint32(D))) | np.uint32(1 << (D - 1))
    pats[:2000] = ties
    pats[2000:4000] = gu.mixed_inputs(2000, 3, fmt).view(np.uint32)
    x = pats.view(np.float32)
    xd = torch.from_numpy(x).cuda()
    for variant in DET:
        for scale in (1.0, 0.75):
            expect = capi.fbsr_round(x, fmt, variant, 1, seed=0, scale=scale)
            gu.assert_codes_equal(fbsr.fbsr_round(xd, fmt, variant, 7, seed=123, offset=5, scale=scale), expect, variant)
            gu.assert_codes_equal(fbsr.fbsr_round(xd[1:], fmt, variant, 3, seed=1, scale=scale), expect[1:], variant + " unaligned")
        codes, st, _, _ = fbsr.fbsr_round_stats(xd, fmt, variant, 2, seed=9)
        ecodes, est, _, _ = capi.fbsr_round_stats(x, fmt, variant, 2, seed=9)
        gu.assert_codes_equal(codes, ecodes, variant + " stats")
        assert st["n_up"] == est["n_up"] and abs(st["sum_e"] - est["sum_e"]) <= 1e-9 * est["sum_abs_e"]
    # nearest-even against torch's own cast on the in-range part
    M = {"bf16": 3.3895313892515355e38, "fp16": 65504.0, "e4m3": 448.0, "e5m2": 57344.0}[fmt]
    ok = torch.isfinite(xd) & (xd.abs() <= M)
    got = fbsr.fbsr_round(xd, fmt, "rtne", 1, seed=0)
    as_int = torch.int16 if got.dtype == torch.uint16 else torch.uint8
    ref = xd.to(TORCH_DTYPE[fmt]).view(as_int)
    assert torch.equal(got.view(as_int)[ok], ref[ok])


@pytest.mark.parametrize("w_fmt", ["e4m3", "e5m2", "b8p4"])
@pytest.mark.parametrize("u_fmt", ["bf16", "fp16"])
def test_qat_update(w_fmt, u_fmt):
    rng = np.random.default_rng(95)
    n = 7 * 1280 + 19
    w8 = rng.integers(0, 256, size=n).astype(np.uint8)                   # every code, NaN/Inf included
    u16 = rng.integers(0, 1 << 16, size=n).astype(np.uint16)
    # most updates small relative to the weight, some arbitrary codes
    wv = np.nan_to_num(capi.decode_array(w_fmt, w8), nan=1.0, posinf=1.0, neginf=-1.0)
    small = (wv * rng.uniform(-0.3, 0.3, n)).astype(np.float32)
    dt = torch.bfloat16 if u_fmt == "bf16" else torch.float16
    small16 = torch.from_numpy(small).to(dt).view(torch.int16).numpy().view(np.uint16)
    u16[: n - 500] = small16[: n - 500]
    # finite sums beyond the 16-bit format's largest value (they saturate; they do not become infinities):
    # the largest finite update code next to weights of the same sign
    top = 0x7F7F if u_fmt == "bf16" else 0x7BFF
    u16[100:164] = np.where(w8[100:164] & 0x80, 0x8000 | top, top).astype(np.uint16)
    for variant, k in (("srff", 3), ("srf", 3), ("src", 3), ("src", 8), ("rtne", 1), ("srf", 16)):
        wd = gu.from_np_codes(w8)
        fbsr.fbsr_qat_update(wd, gu.from_np_codes(u16), w_fmt, u_fmt, variant, k, seed=4, offset=11)
        expect = capi.qat_update(w8.copy(), u16, w_fmt, u_fmt, variant, k, seed=4, offset=11)
        gu.assert_codes_equal(wd, expect, "qat %s<-%s %s k=%d" % (w_fmt, u_fmt, variant, k))


def test_section4_behaviour_in_miniature():
    """Section IV in miniature: precision-4 weights (E4M3), BFloat16 updates, 3 random bits.
    (a) a constant update of 1/16 ulp: round-to-nearest never changes a weight (stagnation);
    (b) updates that leave D = 4 excess bits, all residues equally likely: per step SRFF falls behind the exact
        sum by 2^-5 ulp, SRF runs ahead by 2^-5 ulp, SRC tracks it (Section III-E, III-F at N = 3, D = 4)."""
    n = 1 << 21
    g = torch.Generator(device="cuda").manual_seed(3)
    w_exact = torch.rand(n, generator=g, device="cuda") * 0.25 + 1.0       # [1, 1.25): ulp = 1/8, no binade crossing
    w0 = fbsr.fbsr_round(w_exact, "e4m3", "rtne", 1, seed=0)
    start = w0.view(torch.float8_e4m3fn).double()
    tiny = torch.full((n,), 2.0 ** -7, device="cuda").to(torch.bfloat16).view(torch.uint16)
    w = w0.clone()
    for t in range(8):
        fbsr.fbsr_qat_update(w, tiny, "e4m3", "bf16", "rtne", 1, seed=t)
    assert torch.equal(w, w0)
    steps, ulp = 4, 0.125
    ups = [(torch.randint(0, 16, (n,), generator=g, device="cuda").float() / 128.0) for _ in range(steps)]
    exact = sum(u.double().mean().item() for u in ups)
    gain = {}
    for variant in ("srff", "srf", "src"):
        w = w0.clone()
        for t, u in enumerate(ups):
            fbsr.fbsr_qat_update(w, u.to(torch.bfloat16).view(torch.uint16), "e4m3", "bf16", variant, 3, seed=100 + t)
        gain[variant] = (w.view(torch.float8_e4m3fn).double() - start).mean().item()
    tol = 1.5e-3 * ulp
    assert abs(gain["src"] - exact) < tol
    assert abs(gain["srff"] - (exact - steps * 2.0 ** -5 * ulp)) < tol
    assert abs(gain["srf"] - (exact + steps * 2.0 ** -5 * ulp)) < tol


@pytest.mark.parametrize("fmt", FMTS)
def test_ieee_overflow_option(fmt):
    """FBSR_OVF_IEEE: finite values beyond M follow IEEE nearest-even (M, then Inf / NaN) instead of saturating."""
    rng = np.random.default_rng(97)
    M = np.float32({"bf16": 3.3895313892515355e38, "fp16": 65504.0, "e4m3": 448.0, "e5m2": 57344.0}[fmt])
    n = 6000
    x = (M * (1.0 + rng.uniform(-0.2, 0.2, n))).astype(np.float32) * np.where(rng.integers(0, 2, n), 1, -1).astype(np.float32)
    x[:100] = gu.mixed_inputs(100, 5, fmt)
    P = {"bf16": 8, "fp16": 11, "e4m3": 4, "e5m2": 3}[fmt]
    ulp = np.float32(2.0 ** (np.floor(np.log2(float(M))) - (P - 1)))
    x[100:104] = [M + ulp / 2, -(M + ulp / 2), np.nextafter(np.float32(M + ulp / 2), np.float32(0)), np.nextafter(M, np.float32(np.inf))]
    x = np.where(np.isinf(x), M, x).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    for variant, k in (("rtne", 1), ("srf", 3), ("src", 8)):
        got = fbsr.fbsr_round(xd, fmt + "+ieee", variant, k, seed=2, offset=7)
        gu.assert_codes_equal(got, capi.fbsr_round(x, fmt + "+ieee", variant, k, seed=2, offset=7), fmt + " ieee " + variant)
        codes, st, _, _ = fbsr.fbsr_round_stats(xd, fmt + "+ieee", variant, k, seed=2, offset=7)
        assert torch.equal(codes, got)
    # nearest-even with the flag equals torch's cast on every finite input (torch overflows the same way)
    got = fbsr.fbsr_round(xd, fmt + "+ieee", "rtne", 1, seed=0)
    as_int = torch.int16 if got.dtype == torch.uint16 else torch.uint8
    ref = xd.to(TORCH_DTYPE[fmt]).view(as_int)
    mask = 0x7FFF if got.dtype == torch.uint16 else 0x7F
    ok = torch.isfinite(xd)
    assert torch.equal(got.view(as_int)[ok] & mask, ref[ok] & mask)


def test_ieee_overflow_option_with_supplied_bits_and_16_bit_sources():
    """The same option through fbsr_round_bits and fbsr_round_lp (the tiled IEEE variant for 16-bit sources, the general kernel for supplied bits)."""
    rng = np.random.default_rng(99)
    n = 9 * 1280 + 301
    x = (np.float32(448.0) * (1.0 + rng.uniform(-0.3, 0.3, n))).astype(np.float32) * np.where(rng.integers(0, 2, n), 1, -1).astype(np.float32)
    x[:200] = gu.mixed_inputs(200, 6, "e4m3")
    xd = torch.from_numpy(x).cuda()
    for fmt in ("e4m3", "e5m2", "b8p4"):
        for variant, k in (("srf", 3), ("src", 4)):
            words = capi.random_words(seed=3, offset=0, count=n, k=k)
            got = fbsr.fbsr_round_bits(xd, fmt + "+ieee", variant, k, gu.from_np_u32(words), scale=0.6)
            gu.assert_codes_equal(got, capi.fbsr_round_bits(x, fmt + "+ieee", variant, k, words, scale=0.6), "bits " + fmt)
    codes16 = rng.integers(0, 1 << 16, size=n).astype(np.uint16)          # every kind of bf16 / fp16 code, huge ones included
    cd = gu.from_np_codes(codes16)
    for src_fmt in ("bf16", "fp16"):
        for fmt in ("e4m3", "e5m2", "b8p4"):
            got = fbsr.fbsr_round_lp(cd, src_fmt, fmt + "+ieee", "src", 3, seed=8, offset=2560, scale=1.5)
            gu.assert_codes_equal(got, capi.fbsr_round_lp(codes16, src_fmt, fmt + "+ieee", "src", 3, seed=8, offset=2560, scale=1.5),
                                  "lp %s->%s" % (src_fmt, fmt))
