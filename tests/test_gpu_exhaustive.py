"""Every one of the 2^32 binary32 inputs, for a few (format, variant, k): the GPU result equals the
oracle's.  The oracle side runs on all host cores (disjoint chunks, global index as offset); if the time
budget ever cuts it short, the fraction that ran is printed and raised as a warning."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt,variant,k", [("bf16", "src", 5), ("e4m3", "srf", 3), ("fp16", "src", 13), ("b8p4", "src", 3)])
def test_all_binary32_patterns(fmt, variant, k):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util as gu
    capi.lib()
    chunk = 1 << 28
    base = torch.arange(chunk, dtype=torch.int64, device="cuda")
    out = torch.empty(chunk, dtype=fbsr.CODE_DTYPE[fmt], device="cuda")
    x_pin, xh = gu.pinned_like(torch.empty(chunk, dtype=torch.float32))
    out_pin, got = gu.pinned_like(out)
    chk = gu.WholeTensorChecker(budget_s=150)
    for c in range(16):
        start = c * chunk
        x = (base + start).to(torch.int32).view(torch.float32) if start < 2 ** 31 else \
            (base + (start - 2 ** 32)).to(torch.int32).view(torch.float32)
        fbsr.fbsr_round(x, fmt, variant, k, seed=2024, offset=start, scale=1.0, out=out)
        x_pin.copy_(x)
        out_pin.copy_(out)
        torch.cuda.synchronize()

        def piece(a, b, start=start):
            expect = capi.fbsr_round(xh[a:b], fmt, variant, k, seed=2024, offset=start + a)
            return gu.first_difference(got[a:b], expect, start + a, "binary32 pattern")

        chk.run(chunk, piece, remaining_calls=16 - c)
    chk.report("all 2^32 binary32 patterns, %s %s k=%d" % (fmt, variant, k))
    assert chk.fraction > 0.05
