"""GPU parity for the Binary8P4 target (Section IV's format): what is particular to it -- one zero, one NaN,
infinities at the all-ones magnitude -- through every entry point, and the Section IV setting itself."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import VARIANTS  # noqa: E402

FMT = "b8p4"
ALL_VARIANTS = VARIANTS + ("rtne", "rta", "rto")


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu = fbsr, capi, gpu_util


def decode(codes_t):
    """Values of Binary8P4 codes as float64 on the device (test-side table built from the oracle)."""
    table = torch.from_numpy(capi.decode_array(FMT, np.arange(256, dtype=np.uint8)).astype(np.float64)).cuda()
    return table[codes_t.long()]


def test_zero_results_have_no_sign_and_nan_is_0x80():
    """Dense in the cases that differ from the other formats: values around and below the smallest subnormal
    (2^-10) of both signs, zeros of both signs, NaNs of both signs, infinities, values around M = 224."""
    rng = np.random.default_rng(41)
    n = 9 * 1536 + 5
    mag = rng.choice(np.array([0.0, 2.0 ** -10, 2.0 ** -11, 2.0 ** -12, 3 * 2.0 ** -13, 2.0 ** -20, 2.0 ** -40, 1e-44,
                               224.0, 223.9, 224.1, 231.9, 232.0, 232.1, 240.0, 1e9, np.inf, np.nan, 1.0, 0.0078125]),
                     size=n).astype(np.float32)
    jitter = (1 + rng.integers(-2, 3, size=n) * 2.0 ** -23).astype(np.float32)
    x = (mag * jitter * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=n)).astype(np.float32)
    xd = torch.from_numpy(x).cuda()
    for variant in ALL_VARIANTS:
        for k in (1, 3, 4, 9, 16):
            for fmt in (FMT, FMT + "+ieee"):
                got = fbsr.fbsr_round(xd, fmt, variant, k, seed=8, offset=0)
                gu.assert_codes_equal(got, capi.fbsr_round(x, fmt, variant, k, seed=8, offset=0), "%s %s k=%d" % (fmt, variant, k))
    got = gu.to_np(fbsr.fbsr_round(xd, FMT, "srf", 4, seed=8))
    assert np.all(got[np.isnan(x)] == 0x80) and np.all(got[x == 0] == 0x00)
    assert np.all(got[np.isposinf(x)] == 0x7F) and np.all(got[np.isneginf(x)] == 0xFF)
    tiny_neg = (x < 0) & (x > -2.0 ** -30)
    assert tiny_neg.any() and np.all(got[tiny_neg] == 0x00)               # never 0x80
    assert np.all(got[np.isfinite(x) & (x > 224)] == 0x7E) and np.all(got[np.isfinite(x) & (x < -224)] == 0xFE)


def test_statistics_and_supplied_bits():
    n = 60_000 + 3
    x = gu.mixed_inputs(n, 43, FMT)
    xd = torch.from_numpy(x).cuda()
    for variant, k in (("srff", 3), ("src", 4), ("srf", 7)):
        codes, st, ge, _ = fbsr.fbsr_round_stats(xd, FMT, variant, k, seed=5, offset=9, scale=0.75, group_size=500)
        ecodes, est, ege, _ = capi.fbsr_round_stats(x, FMT, variant, k, seed=5, offset=9, scale=0.75, group_size=500)
        gu.assert_codes_equal(codes, ecodes, "stats codes")
        for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
            assert st[key] == est[key], key
        assert abs(st["sum_e"] - est["sum_e"]) <= 1e-9 * est["sum_abs_e"]
        assert np.allclose(ge.cpu().numpy(), ege, rtol=1e-9, atol=1e-9)
        words = capi.random_words(seed=5, offset=0, count=n, k=k)
        got = fbsr.fbsr_round_bits(xd, FMT, variant, k, gu.from_np_u32(words), scale=0.75)
        gu.assert_codes_equal(got, capi.fbsr_round_bits(x, FMT, variant, k, words, scale=0.75), "bits")


def test_accumulate_and_qat_update_on_every_code():
    """The stored codes include 0x80 (NaN) and 0x7F / 0xFF (infinities), which decode unlike E4M3's."""
    rng = np.random.default_rng(47)
    n = 8 * 2560 + 33
    w8 = np.concatenate([np.arange(256), rng.integers(0, 256, size=n - 256)]).astype(np.uint8)
    vals = np.nan_to_num(capi.decode_array(FMT, w8), nan=1.0, posinf=1.0, neginf=-1.0)
    u = (vals * rng.uniform(-0.2, 0.2, n)).astype(np.float32)
    u[::97] = -vals[::97]                                                   # exact cancellation: a zero result
    for variant, k in (("srff", 3), ("srf", 3), ("src", 3), ("rtne", 1), ("src", 6), ("srf", 10)):
        wd = gu.from_np_codes(w8)
        fbsr.fbsr_accumulate(wd, torch.from_numpy(u).cuda(), FMT, variant, k, seed=3, offset=5)
        expect = capi.accumulate(w8.copy(), u, FMT, variant, k, seed=3, offset=5)
        gu.assert_codes_equal(wd, expect, "accumulate %s k=%d" % (variant, k))
        for u_fmt, dt in (("bf16", torch.bfloat16), ("fp16", torch.float16)):
            u16 = torch.from_numpy(u).to(dt).view(torch.int16).numpy().view(np.uint16).copy()
            u16[-300:] = rng.integers(0, 1 << 16, size=300).astype(np.uint16)      # arbitrary codes too
            wd = gu.from_np_codes(w8)
            fbsr.fbsr_qat_update(wd, gu.from_np_codes(u16), FMT, u_fmt, variant, k, seed=3, offset=5)
            expect = capi.qat_update(w8.copy(), u16, FMT, u_fmt, variant, k, seed=3, offset=5)
            gu.assert_codes_equal(wd, expect, "qat %s %s k=%d" % (u_fmt, variant, k))


def test_section4_setting_with_the_papers_format():
    """Section IV as the paper ran it: Binary8P4 weights, BFloat16 updates, 3 random bits (D = 4 excess bits).
    (a) updates of 1/16 ulp: round-to-nearest never changes a weight (stagnation);
    (b) all 16 residues equally likely: per step SRFF falls behind the exact sum by 2^-5 ulp, SRF runs ahead by
        2^-5 ulp, SRC tracks it (Section III-E and III-F at N = 3, D = 4)."""
    n = 1 << 21
    g = torch.Generator(device="cuda").manual_seed(5)
    w_exact = torch.rand(n, generator=g, device="cuda") * 0.25 + 1.0       # [1, 1.25): ulp = 1/8, no binade crossing
    w0 = fbsr.fbsr_round(w_exact, FMT, "rtne", 1, seed=0)
    start = decode(w0)
    assert float((start - w_exact.double()).abs().max()) <= 0.0625
    tiny = torch.full((n,), 2.0 ** -7, device="cuda").to(torch.bfloat16).view(torch.uint16)
    w = w0.clone()
    for t in range(8):
        fbsr.fbsr_qat_update(w, tiny, FMT, "bf16", "rtne", 1, seed=t)
    assert torch.equal(w, w0)
    steps, ulp = 4, 0.125
    ups = [(torch.randint(0, 16, (n,), generator=g, device="cuda").float() / 128.0) for _ in range(steps)]
    exact = sum(u.double().mean().item() for u in ups)
    gain = {}
    for variant in VARIANTS:
        w = w0.clone()
        for t, u in enumerate(ups):
            before = gu.to_np(w).copy() if t == 0 else None
            u16 = u.to(torch.bfloat16).view(torch.uint16)
            fbsr.fbsr_qat_update(w, u16, FMT, "bf16", variant, 3, seed=100 + t)
            if t == 0:
                e = capi.qat_update(before[:50_000], gu.to_np(u16)[:50_000], FMT, "bf16", variant, 3, seed=100)
                assert np.array_equal(gu.to_np(w)[:50_000], e)
        gain[variant] = (decode(w) - start).mean().item()
    tol = 1.5e-3 * ulp
    assert abs(gain["src"] - exact) < tol
    assert abs(gain["srff"] - (exact - steps * 2.0 ** -5 * ulp)) < tol
    assert abs(gain["srf"] - (exact + steps * 2.0 ** -5 * ulp)) < tol


def test_full_size_launch_on_sampled_slices():
    """2^27 elements in one launch (the fp8 configuration's size), compared on sampled tiles, plus properties
    that hold for every element: no 0x80 from a finite input, magnitudes never beyond M."""
    n = 1 << 27
    g = torch.Generator(device="cuda").manual_seed(13)
    x = torch.empty(n, device="cuda").exponential_(1.0, generator=g)
    x *= torch.where(torch.rand(n, device="cuda", generator=g) < 0.5, -1.0, 1.0)
    for variant, k in (("srf", 3), ("src", 4)):
        got = fbsr.fbsr_round(x, FMT, variant, k, seed=99, scale=24.0)
        assert int((got == 0x80).sum()) == 0 and int(((got & 0x7F) == 0x7F).sum()) == 0
        tile = fbsr.fbsr_tile_elements(k)
        for a in (0, 1000 * tile, n - 3 * tile, (n // 2 // tile) * tile):
            b = min(a + 3 * tile, n)
            e = capi.fbsr_round(x[a:b].cpu().numpy(), FMT, variant, k, seed=99, offset=a, scale=24.0)
            gu.assert_codes_equal(got[a:b], e, "slice at %d" % a)
        err = (decode(got[: 1 << 22]) - (x[: 1 << 22].double() * 24.0).clamp(-224, 224)).abs()
        assert float(err.max()) <= 16.0                                   # never more than one ulp of the top binade
