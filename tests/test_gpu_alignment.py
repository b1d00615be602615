"""The two fast kernels behind fbsr_round for every draw width, format and variant: the aligned tiled kernel and
the staged kernel that takes pointers of any element alignment (codes funnelled to 4-byte words in global
memory, the bytes around a tile's first and last aligned word stored one code at a time), both also with the
IEEE overflow option where it is served by tiles.  Outputs sit between canaries; results are the oracle's bit
for bit and misaligned calls really take the fast kernel (one launch more than the head needs, not a general
launch over the whole call)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import ALL_FMTS, VARIANTS  # noqa: E402


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu = fbsr, capi, gpu_util


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_every_draw_width_on_misaligned_pointers(fmt):
    for k in range(1, 17):
        tile = fbsr.fbsr_tile_elements(k)
        n = 5 * tile + 77
        x = gu.mixed_inputs(n + 8, 900 + k, fmt)
        xd = torch.from_numpy(x).cuda()
        variant = VARIANTS[k % 3]
        for skip_in, skip_out in ((1, 0), (0, 1), (5, 3), (2, 2), (7, 6)):
            raw, out = gu.guarded(n, fbsr.CODE_DTYPE[fmt], misalign=skip_out)
            src = xd[skip_in: skip_in + n]
            fbsr.fbsr_round(src, fmt, variant, k, seed=31, offset=3 * tile, scale=1.5, out=out)
            torch.cuda.synchronize()
            expect = capi.fbsr_round(x[skip_in: skip_in + n], fmt, variant, k, seed=31, offset=3 * tile, scale=1.5)
            gu.assert_codes_equal(out, expect, "%s %s k=%d skip=%d/%d" % (fmt, variant, k, skip_in, skip_out))
            assert gu.canaries_intact(raw, n, fbsr.CODE_DTYPE[fmt], misalign=skip_out)


def test_misaligned_calls_take_one_launch():
    """offset on the tile grid: a misaligned call is one launch of the staged kernel (tiles and ragged end)."""
    x = torch.from_numpy(gu.mixed_inputs(40_000, 1, "bf16")).cuda()
    for fmt in ("bf16", "e4m3"):
        out = torch.empty(39_990, dtype=fbsr.CODE_DTYPE[fmt], device="cuda")
        before = fbsr.fbsr_launch_count()
        fbsr.fbsr_round(x[3:39_993], fmt, "srf", 4, seed=1, offset=0, out=out)
        assert fbsr.fbsr_launch_count() - before == 1


@pytest.mark.parametrize("fmt", ALL_FMTS)
def test_ieee_overflow_on_whole_tiles_for_every_draw_width(fmt):
    M = {"bf16": 3.3895313892515355e38, "fp16": 65504.0, "e4m3": 448.0, "e5m2": 57344.0, "b8p4": 224.0}[fmt]
    rng = np.random.default_rng(5)
    for k in range(1, 17):
        tile = fbsr.fbsr_tile_elements(k)
        n = 4 * tile + 13
        x = gu.mixed_inputs(n, 700 + k, fmt)
        # a third of the elements around M: below, on and beyond the midpoint to the next power of two
        pos = rng.choice(n, size=n // 3, replace=False)
        x[pos] = (np.float32(M) * (1.0 + rng.uniform(-0.1, 0.1, pos.size))).astype(np.float32) * rng.choice([-1.0, 1.0], pos.size).astype(np.float32)
        x = np.where(np.isinf(x), np.float32(M), x).astype(np.float32)
        xd = torch.from_numpy(x).cuda()
        for variant in VARIANTS:
            got = fbsr.fbsr_round(xd, fmt + "+ieee", variant, k, seed=9, offset=2 * tile)
            gu.assert_codes_equal(got, capi.fbsr_round(x, fmt + "+ieee", variant, k, seed=9, offset=2 * tile),
                                  "%s ieee %s k=%d" % (fmt, variant, k))


def test_an_lp_call_aligned_as_documented_takes_the_tiled_path():
    """fbsr_round_lp: source 32-byte aligned, codes 16-byte aligned, offset on the tile grid -> one launch of the tiled
    kernel for the whole call; a source that is only 16-byte aligned falls to the general kernel, still one launch, and
    gives the same codes."""
    tile = 2 * fbsr.fbsr_tile_elements(3)                 # 16 codes per lane: the tiles of this entry point are twice as long
    n = 6 * tile + 5
    codes = torch.randint(0, 1 << 15, (n + 16,), device="cuda", dtype=torch.int32).to(torch.uint16)
    assert codes.data_ptr() % 32 == 0
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    before = fbsr.fbsr_launch_count()
    fbsr.fbsr_round_lp(codes[:n], "bf16", "e4m3", "src", 3, seed=4, offset=3 * tile, out=out)
    assert fbsr.fbsr_launch_count() - before == 1
    expect = capi.fbsr_round_lp(gu.to_np(codes[:n]), "bf16", "e4m3", "src", 3, seed=4, offset=3 * tile)
    gu.assert_codes_equal(out, expect, "aligned lp call")
    out2 = torch.empty(n, dtype=torch.uint8, device="cuda")
    fbsr.fbsr_round_lp(codes[8:8 + n], "bf16", "e4m3", "src", 3, seed=4, offset=3 * tile, out=out2)      # 16 bytes off
    gu.assert_codes_equal(out2, capi.fbsr_round_lp(gu.to_np(codes[8:8 + n]), "bf16", "e4m3", "src", 3, seed=4, offset=3 * tile),
                          "lp call 16 bytes off")
