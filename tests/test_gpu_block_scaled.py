"""GPU parity for block-scaled rounding (fbsr_round_mx): codes and scale bytes against the oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import ALL_FMTS as FMTS, VARIANTS  # noqa: E402


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from paper_2504_20634_b200 import workloads
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu, module.workloads = fbsr, capi, gpu_util, workloads


@pytest.mark.parametrize("fmt", FMTS)
def test_block_scaled_parity(fmt):
    rng = np.random.default_rng(60 + FMTS.index(fmt))
    for k, variant in ((2, "srff"), (3, "src"), (4, "srf"), (8, "src"), (13, "srf"), (1, "rtne")):
        tile = fbsr.fbsr_tile_elements(k)
        n = 7 * tile + 45                                       # ragged last block
        x = gu.mixed_inputs(n, 600 + k, fmt)
        x[256:320] = 0.0                                        # all-zero blocks
        x[320:352] = rng.integers(0, 1 << 23, size=32, dtype=np.uint32).view(np.float32)   # subnormal-only block
        x[352:384] = np.float32(np.inf)                         # a block without finite values
        xd = torch.from_numpy(x).cuda()
        for offset in (0, 3 * tile, 5):                         # 5: the first tile boundary is off the block grid
            raw, out = gu.guarded(n, fbsr.CODE_DTYPE[fmt])
            sraw, sc = gu.guarded((n + 31) // 32, torch.uint8)
            fbsr.fbsr_round_mx(xd, fmt, variant, k, seed=17, offset=offset, out=out, scales=sc)
            torch.cuda.synchronize()
            ecodes, escales = capi.fbsr_round_mx(x, fmt, variant, k, seed=17, offset=offset)
            assert np.array_equal(sc.cpu().numpy(), escales), "scales k=%d offset=%d" % (k, offset)
            gu.assert_codes_equal(out, ecodes, "mx %s %s k=%d offset=%d" % (fmt, variant, k, offset))
            assert gu.canaries_intact(raw, n, fbsr.CODE_DTYPE[fmt]) and gu.canaries_intact(sraw, (n + 31) // 32, torch.uint8)
        # unaligned source: the general kernel
        out, sc = fbsr.fbsr_round_mx(xd[1:], fmt, variant, k, seed=17)
        ecodes, escales = capi.fbsr_round_mx(x[1:], fmt, variant, k, seed=17)
        assert np.array_equal(sc.cpu().numpy(), escales)
        gu.assert_codes_equal(out, ecodes, "mx unaligned")


def test_block_scaled_large_sampled():
    n = 1 << 27
    x = workloads.bandwidth_sweep(n, seed=1234, device="cuda")
    out, sc = fbsr.fbsr_round_mx(x, "e4m3", "src", 3, seed=5)
    rng = np.random.default_rng(9)
    for a in [0, n - 8192] + [int(s) * 32 for s in rng.integers(0, (n - 8192) // 32, size=6)]:
        ecodes, escales = capi.fbsr_round_mx(x[a:a + 8192].cpu().numpy(), "e4m3", "src", 3, seed=5, offset=a)
        gu.assert_codes_equal(out[a:a + 8192], ecodes, "mx large at %d" % a)
        assert np.array_equal(sc[a // 32:(a + 8192) // 32].cpu().numpy(), escales)
