"""Every one of the 2^32 binary32 inputs, for a few (format, variant, k): the GPU result equals the
oracle's.  The oracle side runs on all host cores (disjoint chunks, global index as offset)."""
import concurrent.futures
import os

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
    threads = max(1, min(32, os.cpu_count() or 1))
    # with few host cores only every 16th block of 2^20 patterns is checked by the oracle
    stride = 1 if threads >= 8 else 16
    chunk = 1 << 28
    piece = 1 << 20
    base = torch.arange(chunk, dtype=torch.int64, device="cuda")
    out = torch.empty(chunk, dtype=fbsr.CODE_DTYPE[fmt], device="cuda")
    with concurrent.futures.ThreadPoolExecutor(threads) as pool:
        for c in range(16):
            start = c * chunk
            x = (base + start).to(torch.int32).view(torch.float32) if start < 2 ** 31 else \
                (base + (start - 2 ** 32)).to(torch.int32).view(torch.float32)
            fbsr.fbsr_round(x, fmt, variant, k, seed=2024, offset=start, scale=1.0, out=out)
            got = gu.to_np(out)
            xh = x.cpu().numpy()

            def check(j):
                a, b = j * piece, (j + 1) * piece
                expect = capi.fbsr_round(xh[a:b], fmt, variant, k, seed=2024, offset=start + a)
                if not np.array_equal(got[a:b], expect):
                    bad = np.nonzero(got[a:b] != expect)[0][0]
                    return "pattern %#010x: got %#x expect %#x" % (start + a + bad, got[a + bad], expect[bad])
                return None

            for res in pool.map(check, range(0, chunk // piece, stride)):
                assert res is None, res
