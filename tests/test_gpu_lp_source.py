"""GPU parity for 16-bit sources rounded to 8-bit formats (fbsr_round_lp), and the Fig. 2 experiment."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import VARIANTS  # noqa: E402


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from paper_2504_20634_b200 import workloads
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu, module.workloads = fbsr, capi, gpu_util, workloads


@pytest.mark.parametrize("src_fmt", ["bf16", "fp16"])
@pytest.mark.parametrize("dst_fmt", ["e4m3", "e5m2", "b8p4"])
def test_every_source_code_every_k(src_fmt, dst_fmt):
    """All 65536 source codes (NaN, Inf, subnormals, saturating values included), shuffled and tiled so that
    several tiles and a ragged tail are covered, every k and variant."""
    rng = np.random.default_rng(5)
    codes = np.concatenate([rng.permutation(1 << 16), rng.integers(0, 1 << 16, size=1237)]).astype(np.uint16)
    cd = gu.from_np_codes(codes)
    for k in range(1, 17):
        for variant in VARIANTS:
            scale = 1.0 if k % 3 else 0.6
            raw, out = gu.guarded(codes.size, torch.uint8)
            fbsr.fbsr_round_lp(cd, src_fmt, dst_fmt, variant, k, seed=31 + k, offset=0, scale=scale, out=out)
            torch.cuda.synchronize()
            expect = capi.fbsr_round_lp(codes, src_fmt, dst_fmt, variant, k, seed=31 + k, offset=0, scale=scale)
            gu.assert_codes_equal(out, expect, "%s->%s %s k=%d" % (src_fmt, dst_fmt, variant, k))
            assert gu.canaries_intact(raw, codes.size, torch.uint8)


def test_offsets_and_alignment():
    rng = np.random.default_rng(6)
    codes = rng.integers(0, 1 << 16, size=20_011).astype(np.uint16)
    cd = gu.from_np_codes(codes)
    for k in (2, 3, 8):
        for offset in (0, 7, 5 * fbsr.fbsr_tile_elements(k), 2 ** 41 + 3):
            for skip in (0, 1, 5):
                n = codes.size - 8
                raw, out = gu.guarded(n, torch.uint8, misalign=skip)
                fbsr.fbsr_round_lp(cd[skip:skip + n], "bf16", "e4m3", "srf", k, seed=2, offset=offset, out=out)
                torch.cuda.synchronize()
                gu.assert_codes_equal(out, capi.fbsr_round_lp(codes[skip:skip + n], "bf16", "e4m3", "srf", k, seed=2, offset=offset),
                                      "k=%d offset=%d skip=%d" % (k, offset, skip))
                assert gu.canaries_intact(raw, n, torch.uint8, misalign=skip)
    for bad in (("fp16", "bf16"), ("e4m3", "e5m2"), ("bf16", "fp16")):
        with pytest.raises(fbsr.FbsrError) as err:
            fbsr.fbsr_round_lp(cd, bad[0], bad[1], "srf", 3, seed=0,
                               out=torch.empty(codes.size, dtype=fbsr.CODE_DTYPE[bad[1]], device="cuda"))
        assert err.value.status == 2


def test_fig2_experiment_on_gpu():
    """Fig. 2: every BFloat16 X of [1, 2) sampled 100 000 times, 3 random bits, precision-3 target.
    Codes bit-exact against the oracle; bias -0.046875 / +0.015625 / 0.000 within sampling error."""
    codes = workloads.fig2_grid(device="cuda")
    ch = gu.to_np(codes)
    x = codes.view(torch.bfloat16).double()
    for variant, expect in (("srff", -0.046875), ("srf", 0.015625), ("src", 0.0)):
        out = fbsr.fbsr_round_lp(codes, "bf16", "e5m2", variant, 3, seed=0)
        gu.assert_codes_equal(out, capi.fbsr_round_lp(ch, "bf16", "e5m2", variant, 3, seed=0), "fig2 " + variant)
        bias = ((out.view(torch.float8_e5m2).double() - x) / 0.25).mean().item()
        assert abs(bias - expect) < 5e-4, (variant, bias)


def test_large_lp_sweep_sampled():
    """2^28 BFloat16 codes to both 8-bit formats, sampled slices against the oracle."""
    n = 1 << 28
    codes = workloads.lp_sweep(n, "bf16", device="cuda")
    rng = np.random.default_rng(8)
    slices = [(0, 8192), (n - 8192, n)] + [(int(s), int(s) + 8192) for s in rng.integers(0, n - 8192, size=6)]
    hs = [gu.to_np(codes[a:b]) for a, b in slices]
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    for dst_fmt in ("e4m3", "e5m2"):
        for variant, k in (("srff", 2), ("srf", 3), ("src", 4), ("src", 3), ("srf", 8)):
            fbsr.fbsr_round_lp(codes, "bf16", dst_fmt, variant, k, seed=5, out=out)
            for (a, b), h in zip(slices, hs):
                gu.assert_codes_equal(out[a:b], capi.fbsr_round_lp(h, "bf16", dst_fmt, variant, k, seed=5, offset=a),
                                      "%s %s k=%d at %d" % (dst_fmt, variant, k, a))


@pytest.mark.parametrize("src_fmt", ["bf16", "fp16"])
def test_power_of_two_scales_with_nearest_first_variants(src_fmt):
    """With a power-of-two scale the kernels that round to nearest first (SRC, ties to even / odd) drop the sticky
    bit, because a 16-bit value loses bits in the rescaled pattern only far below every tie: every source code, scales
    that push the values deep below and far above the targets' ranges (and into binary32's own subnormals)."""
    codes = np.arange(1 << 16, dtype=np.uint16)
    cd = gu.from_np_codes(codes)
    for dst_fmt in ("e4m3", "e5m2", "b8p4"):
        for scale in (2.0 ** -30, 2.0 ** -13, 2.0 ** -7, 0.5, 2.0 ** 9, 2.0 ** 40, 2.0 ** -120):
            for variant, k in (("src", 1), ("src", 3), ("src", 8), ("src", 12), ("src", 13), ("src", 16), ("rtne", 1), ("rto", 1)):
                got = fbsr.fbsr_round_lp(cd, src_fmt, dst_fmt, variant, k, seed=77, offset=0, scale=scale)
                expect = capi.fbsr_round_lp(codes, src_fmt, dst_fmt, variant, k, seed=77, offset=0, scale=scale)
                gu.assert_codes_equal(got, expect, "%s->%s %s k=%d scale=%g" % (src_fmt, dst_fmt, variant, k, scale))
