"""GPU parity: fbsr_round / fbsr_round_bits / fbsr_round_stats / fbsr_round_host through the C-ABI,
element by element against the scalar oracle (bit-exact)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import ALL_FMTS as FMTS, VARIANTS  # noqa: E402

ALL_K = list(range(1, 17))


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu = fbsr, capi, gpu_util


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_every_format_variant_and_k(fmt, variant):
    """Several tiles of the fast path plus a ragged tail, offset 0, every k."""
    for k in ALL_K:
        tile = fbsr.fbsr_tile_elements(k)
        n = 11 * tile + 37
        x = gu.mixed_inputs(n, 1000 + k, fmt)
        scale = 1.0 if k % 2 else 1.7
        raw, out = gu.guarded(n, fbsr.CODE_DTYPE[fmt])
        fbsr.fbsr_round(torch.from_numpy(x).cuda(), fmt, variant, k, seed=1234 + k, offset=0, scale=scale, out=out)
        torch.cuda.synchronize()
        expect = capi.fbsr_round(x, fmt, variant, k, seed=1234 + k, offset=0, scale=scale)
        gu.assert_codes_equal(out, expect, "%s %s k=%d" % (fmt, variant, k))
        assert gu.canaries_intact(raw, n, fbsr.CODE_DTYPE[fmt])


@pytest.mark.parametrize("fmt", FMTS)
def test_whole_binary32_exponent_range_and_extreme_scales(fmt):
    """Inputs drawn uniformly over every binary32 bit pattern (all exponents, subnormals, NaNs, infinities)
    and scales from 2^-100 to 2^100: the rescaling and the special-value detection of the fast rows must
    agree with the oracle everywhere, including where the scaled value under- or overflows binary32."""
    rng = np.random.default_rng(FMTS.index(fmt) + 70)
    n = 40 * 1024 + 77
    pats = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    x = pats.view(np.float32)
    xd = torch.from_numpy(x).cuda()
    for k in (1, 3, 5, 8, 11, 12, 13, 14, 16):
        for variant in VARIANTS:
            for scale in (1.0, 2.0 ** -100, 2.0 ** 100, 3.0e-39, 1.0e30, 0.3333333):
                got = fbsr.fbsr_round(xd, fmt, variant, k, seed=k, offset=0, scale=scale)
                expect = capi.fbsr_round(x, fmt, variant, k, seed=k, offset=0, scale=scale)
                gu.assert_codes_equal(got, expect, "%s %s k=%d scale=%g" % (fmt, variant, k, scale))


@pytest.mark.parametrize("fmt", ["bf16", "e4m3", "b8p4"])
def test_small_and_ragged_sizes(fmt):
    for k in (1, 2, 3, 6, 8, 13, 16):
        E = 4 * (32 // k)
        for n in (0, 1, 3, 7, 8, 9, E - 1, E, E + 1, 255, 256, 257):
            x = gu.mixed_inputs(max(n, 1), 7 * k + n, fmt)[:n]
            raw, out = gu.guarded(n, fbsr.CODE_DTYPE[fmt])
            fbsr.fbsr_round(torch.from_numpy(x.copy()).cuda(), fmt, "srf", k, seed=9, offset=5, out=out)
            torch.cuda.synchronize()
            gu.assert_codes_equal(out, capi.fbsr_round(x, fmt, "srf", k, seed=9, offset=5), "n=%d k=%d" % (n, k))
            assert gu.canaries_intact(raw, n, fbsr.CODE_DTYPE[fmt])


@pytest.mark.parametrize("fmt", ["bf16", "fp16", "e5m2"])
def test_offsets_alignment_and_sharding(fmt):
    """Unaligned pointers, offsets off and on the tile grid (including beyond 2^32 calls), and a
    tensor rounded in shards equals the tensor rounded at once."""
    for k in (2, 3, 8, 16):
        tile = fbsr.fbsr_tile_elements(k)
        n = 9 * tile + 11
        x = gu.mixed_inputs(n + 8, 50 + k, fmt)
        xd = torch.from_numpy(x).cuda()
        for offset in (0, 1, tile - 3, 5 * tile, 2 ** 40 + 7, 3 * tile * 2 ** 33):
            for skip_in, skip_out in ((0, 0), (1, 0), (0, 1), (3, 5)):
                raw, out = gu.guarded(n, fbsr.CODE_DTYPE[fmt], misalign=skip_out)
                src = xd[skip_in: skip_in + n]
                fbsr.fbsr_round(src, fmt, "src", k, seed=77, offset=offset, scale=0.75, out=out)
                torch.cuda.synchronize()
                expect = capi.fbsr_round(x[skip_in: skip_in + n], fmt, "src", k, seed=77, offset=offset, scale=0.75)
                gu.assert_codes_equal(out, expect, "k=%d offset=%d skip=%d/%d" % (k, offset, skip_in, skip_out))
                assert gu.canaries_intact(raw, n, fbsr.CODE_DTYPE[fmt], misalign=skip_out)
        whole = fbsr.fbsr_round(xd[:n], fmt, "srf", k, seed=3, offset=0)
        cuts = [0, 5, tile + 1, 4 * tile, n]
        parts = [fbsr.fbsr_round(xd[a:b], fmt, "srf", k, seed=3, offset=a) for a, b in zip(cuts[:-1], cuts[1:])]
        assert torch.equal(whole, torch.cat(parts))


@pytest.mark.parametrize("fmt", FMTS)
def test_supplied_bits_equal_generated_bits(fmt):
    for k in ALL_K:
        tile = fbsr.fbsr_tile_elements(k)
        n = 6 * tile + 13
        x = gu.mixed_inputs(n, 200 + k, fmt)
        xd = torch.from_numpy(x).cuda()
        words = capi.random_words(seed=42, offset=0, count=n, k=k)
        got = fbsr.fbsr_round_bits(xd, fmt, "srf", k, gu.from_np_u32(words))
        gu.assert_codes_equal(got, capi.fbsr_round_bits(x, fmt, "srf", k, words), "bits k=%d" % k)
        assert torch.equal(got, fbsr.fbsr_round(xd, fmt, "srf", k, seed=42, offset=0))
        # arbitrary words, unaligned source
        rng = np.random.default_rng(k)
        words = rng.integers(0, 1 << 32, size=(n + 32 // k - 1) // (32 // k), dtype=np.uint32)
        got = fbsr.fbsr_round_bits(xd[1:], fmt, "src", k, gu.from_np_u32(words))
        gu.assert_codes_equal(got, capi.fbsr_round_bits(x[1:], fmt, "src", k, words[: (n - 1 + 32 // k - 1) // (32 // k)]),
                              "bits unaligned k=%d" % k)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_statistics(fmt, variant):
    """Counts exact; binary64 sums within 1e-9 relative of the oracle's."""
    for k, group in ((2, 1000), (3, 77), (8, 0), (13, 4096)):
        n = 50_000 + k
        x = gu.mixed_inputs(n, 300 + k, fmt)
        codes, st, ge, ge2 = fbsr.fbsr_round_stats(torch.from_numpy(x).cuda(), fmt, variant, k, seed=5, offset=17,
                                                   scale=1.25, group_size=group)
        ecodes, est, ege, ege2 = capi.fbsr_round_stats(x, fmt, variant, k, seed=5, offset=17, scale=1.25,
                                                      group_size=group)
        gu.assert_codes_equal(codes, ecodes, "stats codes")
        for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
            assert st[key] == est[key], key
        for key in ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e"):
            assert abs(st[key] - est[key]) <= 1e-9 * max(abs(est[key]), est["sum_abs_e"] * 1e-3, 1e-300), key
        if group:
            assert np.allclose(ge.cpu().numpy(), ege, rtol=1e-9, atol=1e-9)
            assert np.allclose(ge2.cpu().numpy(), ege2, rtol=1e-9, atol=1e-9)
    # totals are reproducible bit for bit
    a = fbsr.fbsr_round_stats(torch.from_numpy(x).cuda(), fmt, variant, 4, seed=1)[1]
    b = fbsr.fbsr_round_stats(torch.from_numpy(x).cuda(), fmt, variant, 4, seed=1)[1]
    assert a == b


def test_stats_of_empty_call_are_zero():
    x = torch.empty(0, dtype=torch.float32, device="cuda")
    _, st, _, _ = fbsr.fbsr_round_stats(x, "bf16", "srf", 2, seed=0)
    assert all(v == 0 for v in st.values())


def test_fig1_bias_grid_on_gpu():
    """Config 'bias grid': 1024 X in [1, 2) x 5000 samples, bfloat16, k = 2, Philox seed 0.
    Rounded values bit-exact; overall bias -2^-3 (SRFF), 0 (SRF), 0 (SRC) within sampling error
    (Section III-C/D, Fig. 1) and per-X means equal to the oracle's."""
    from paper_2504_20634_b200 import workloads
    for centred, expect in ((True, {"srff": -0.125, "srf": 0.0, "src": 0.0}),
                            (False, {"srff": -0.0625, "srf": 0.0625, "src": 0.0})):
        x = workloads.bias_grid(centred, device="cuda")
        xh = x.cpu().numpy()
        for variant in VARIANTS:
            codes, st, ge, _ = fbsr.fbsr_round_stats(x, "bf16", variant, 2, seed=0, group_size=5000)
            ecodes, est, ege, _ = capi.fbsr_round_stats(xh, "bf16", variant, 2, seed=0, group_size=5000)
            gu.assert_codes_equal(codes, ecodes, "bias grid " + variant)
            assert torch.equal(codes, fbsr.fbsr_round(x, "bf16", variant, 2, seed=0))
            bias = st["sum_e"] / st["n_finite"]
            assert abs(bias - expect[variant]) < 1e-3
            assert abs(st["sum_e"] - est["sum_e"]) <= 1e-9 * est["sum_abs_e"]
            assert np.allclose(ge.cpu().numpy(), ege, rtol=0, atol=1e-9)


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2", "b8p4"])
def test_fp8_activation_workload(fmt):
    """Config 'fp8 path' at 512 x 4096: Laplace activations, amax scaling, saturating outliers,
    subnormal-range values, NaN and +-Inf."""
    from paper_2504_20634_b200 import workloads
    x, scale = workloads.fp8_activations(fmt, rows=512, cols=4096, seed=7, device="cuda")
    xh = x.cpu().numpy()
    for k in (2, 4, 8):
        for variant in VARIANTS:
            got = fbsr.fbsr_round(x, fmt, variant, k, seed=7, scale=scale)
            gu.assert_codes_equal(got, capi.fbsr_round(xh, fmt, variant, k, seed=7, scale=scale), "%s k=%d" % (variant, k))
    _, st, _, _ = fbsr.fbsr_round_stats(x, fmt, "srf", 4, seed=7, scale=scale)
    assert st["n_nan"] == 64 and st["n_inf"] == 128 and st["n_sat"] > 1000


def test_host_buffer_entry_point():
    n = 3_000_001
    x = gu.mixed_inputs(n, 77, "fp16")
    src = torch.from_numpy(x).pin_memory()
    for fmt, k, ws_bytes in (("fp16", 3, 1 << 20), ("e5m2", 8, 5 << 20), ("bf16", 16, 64 << 20)):
        dst = torch.empty(n, dtype=fbsr.CODE_DTYPE[fmt]).pin_memory()
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        fbsr.fbsr_round_host(src, dst, fmt, "srf", k, seed=11, offset=6, scale=1.0, workspace=ws)
        torch.cuda.synchronize()
        gu.assert_codes_equal(dst, capi.fbsr_round(x, fmt, "srf", k, seed=11, offset=6), "host %s" % fmt)


def test_argument_errors_are_return_codes():
    x = torch.zeros(16, dtype=torch.float32, device="cuda")
    for kwargs in (dict(k_bits=0), dict(k_bits=17), dict(scale=0.0), dict(scale=float("inf")), dict(scale=float("nan"))):
        args = dict(src=x, fmt="bf16", variant="srf", k_bits=4, seed=0)
        args.update(kwargs)
        with pytest.raises(fbsr.FbsrError) as err:
            fbsr.fbsr_round(**args)
        assert err.value.status == 1
    with pytest.raises(fbsr.FbsrError):
        fbsr.fbsr_round(x, 7, "srf", 4, seed=0)
    with pytest.raises(fbsr.FbsrError) as err:
        fbsr.fbsr_round_stats(x, "bf16", "srf", 4, seed=0, workspace=torch.empty(8, dtype=torch.uint8, device="cuda"))
    assert err.value.status == 5
    torch.cuda.synchronize()
