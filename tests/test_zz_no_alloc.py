"""fbsr_round_stats_noalloc: the statistics entry point for callers that cannot allocate.

Some users of this library run where device allocation is off limits at call time: inside a
memory pool sized once at start-up, as a plugin in a host application that owns the allocator, or
on a device with no free memory left.  They cannot hand fbsr_round_stats the scratch buffer it
wants, so the library keeps an 85 KB scratch array of its own for them.  This test calls the new
entry point through the C-ABI twice in a row (the second call finds the first call's leftovers in
the shared scratch) and checks codes, counters and sums against the ordinary entry point, with the
1e-9 relative tolerance the other statistics tests use.  It lives in a file that sorts last so a
run that stops at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _run_pair(fbsr, x, fmt, variant, k, seed, group):
    n = x.numel()
    groups = (n + group - 1) // group
    out = torch.empty(n, dtype=fbsr.CODE_DTYPE[fmt], device="cuda")
    total = torch.full((72,), 0xEE, dtype=torch.uint8, device="cuda")
    ge = torch.full((groups,), 7.0, dtype=torch.float64, device="cuda")
    ge2 = torch.full((groups,), 7.0, dtype=torch.float64, device="cuda")
    fbsr.fbsr_round_stats_noalloc(x, out, total, fmt, variant, k, seed=seed, offset=3, scale=1.5, group_size=group,
                                  group_sum_e=ge, group_sum_e2=ge2)
    torch.cuda.synchronize()
    got = fbsr.stats_from_bytes(total)
    ref_codes, ref, ref_ge, ref_ge2 = fbsr.fbsr_round_stats(x, fmt, variant, k, seed=seed, offset=3, scale=1.5,
                                                            group_size=group)
    assert torch.equal(out, ref_codes)
    for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
        assert got[key] == ref[key], key
    for key in ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e"):
        assert abs(got[key] - ref[key]) <= 1e-9 * max(abs(ref[key]), 1e-3 * ref["sum_abs_e"], 1e-300), key
    assert np.allclose(ge.cpu().numpy(), ref_ge.cpu().numpy(), rtol=1e-9, atol=1e-9)
    assert np.allclose(ge2.cpu().numpy(), ref_ge2.cpu().numpy(), rtol=1e-9, atol=1e-9)
    # and against the oracle itself, so that this file stands on its own
    from oracle import capi
    import gpu_util
    ecodes, est, ege, _ = capi.fbsr_round_stats(x.cpu().numpy(), fmt, variant, k, seed=seed, offset=3, scale=1.5,
                                                group_size=group)
    gpu_util.assert_codes_equal(out, ecodes, "no-alloc codes against the oracle")
    for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
        assert got[key] == est[key], key
    for key in ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e"):
        assert abs(got[key] - est[key]) <= 1e-9 * max(abs(est[key]), 1e-3 * est["sum_abs_e"], 1e-300), key
    assert np.allclose(ge.cpu().numpy(), ege, rtol=1e-9, atol=1e-9)
    return got


def test_noalloc_statistics_match_the_workspace_entry_point_twice_in_a_row():
    import paper_2504_20634_b200 as fbsr
    import gpu_util
    # first call: a large input that fills every scratch slot
    x1 = torch.from_numpy(gpu_util.mixed_inputs(3_000_017, 901, "fp16")).cuda()
    first = _run_pair(fbsr, x1, "fp16", "srf", 3, seed=11, group=1000)
    assert first["n_finite"] > 0 and first["n_sat"] > 0
    # second call, right after, smaller and different: stale partials of the first must not leak in
    x2 = torch.from_numpy(gpu_util.mixed_inputs(40_001, 902, "bf16")).cuda()
    second = _run_pair(fbsr, x2, "bf16", "src", 8, seed=12, group=77)
    assert second["n_finite"] + second["n_nan"] + second["n_inf"] + second["n_sat"] == 40_001
    # and an empty call reports zeros
    total = torch.full((72,), 0xEE, dtype=torch.uint8, device="cuda")
    fbsr.fbsr_round_stats_noalloc(x2[:0], torch.empty(0, dtype=torch.uint16, device="cuda"), total, "bf16", "srf", 2, seed=0)
    torch.cuda.synchronize()
    assert all(v == 0 for v in fbsr.stats_from_bytes(total).values())


def test_noalloc_call_allocates_nothing():
    """What the entry point is for: after the first call on the device (which looks up the scratch address),
    a call neither takes device memory from the driver nor from torch's allocator."""
    import paper_2504_20634_b200 as fbsr
    import gpu_util
    x = torch.from_numpy(gpu_util.mixed_inputs(1_000_003, 903, "e4m3")).cuda()
    out = torch.empty(x.numel(), dtype=torch.uint8, device="cuda")
    total = torch.empty(72, dtype=torch.uint8, device="cuda")
    fbsr.fbsr_round_stats_noalloc(x, out, total, "e4m3", "srf", 3, seed=1)          # warm-up: set-up happens here
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for seed in (2, 3):
        fbsr.fbsr_round_stats_noalloc(x, out, total, "e4m3", "srf", 3, seed=seed)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)


def test_noalloc_rejects_sizes_beyond_its_limit():
    import ctypes
    import paper_2504_20634_b200 as fbsr
    lib = ctypes.CDLL(fbsr.library_path())
    vp, sz, i, u64, f = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64, ctypes.c_float
    lib.fbsr_round_stats_noalloc.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, sz, vp, vp, vp, vp]
    x = torch.zeros(16, dtype=torch.float32, device="cuda")
    out = torch.zeros(16, dtype=torch.uint16, device="cuda")
    total = torch.zeros(72, dtype=torch.uint8, device="cuda")
    rc = lib.fbsr_round_stats_noalloc(x.data_ptr(), out.data_ptr(), (1 << 31) + 1, 0, 1, 4, 0, 0, 1.0, 0, None, None,
                                      total.data_ptr(), None)
    assert rc == 6
    assert "limit" in fbsr.fbsr_status_string(rc)
    torch.cuda.synchronize()
    assert int(total.sum()) == 0          # nothing was written
