"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the oracle
checks sampled slices element by element (each output is a pure function of the input element and
its global index), and whole-tensor properties that hold at any size are checked with torch."""
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


def _slices(n, width, count, seed):
    rng = np.random.default_rng(seed)
    starts = [0, n - width] + [int(s) for s in rng.integers(0, n - width, size=count - 2)]
    return [(s, s + width) for s in starts]


def test_bandwidth_sweep_full_size():
    """2^28 elements, every (format, variant, k) of the sweep; 10 slices of 8192 elements each,
    including the first and the last (the ragged tail of the 1280-element tiles)."""
    n = 1 << 28
    x = workloads.bandwidth_sweep(n, seed=1234, device="cuda")
    out = torch.empty(n, dtype=torch.uint16, device="cuda")
    slices = _slices(n, 8192, 10, 3)
    xs = [x[a:b].cpu().numpy() for a, b in slices]
    for fmt in ("bf16", "fp16"):
        for variant in VARIANTS:
            for k in (1, 2, 3, 4, 6, 8, 13, 16):
                out.zero_()
                fbsr.fbsr_round(x, fmt, variant, k, seed=1234, offset=0, out=out)
                for (a, b), xh in zip(slices, xs):
                    expect = capi.fbsr_round(xh, fmt, variant, k, seed=1234, offset=a)
                    gu.assert_codes_equal(out[a:b], expect, "%s %s k=%d slice %d" % (fmt, variant, k, a))
                if fmt == "bf16" and k in (2, 16):
                    # Eq. (5) on the whole tensor: the code is the truncated pattern or its successor,
                    # and exactly representable inputs are unchanged.
                    bits = x.view(torch.int32)
                    lo = (bits >> 16) & 0xFFFF
                    got = out.view(torch.int16).to(torch.int32) & 0xFFFF
                    up = got - lo
                    assert bool(((up == 0) | (up == 1)).all())
                    exact = (bits & 0xFFFF) == 0
                    assert bool((up[exact] == 0).all())
                    if k == 16 and variant == "srff":
                        # with all 16 bits the round-up frequency equals the mean fractional part
                        frac = ((bits & 0xFFFF).double() / 65536.0).mean().item()
                        assert abs(up.double().mean().item() - frac) < 2e-4
                    del bits, lo, got, up, exact


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_activations_full_size(fmt):
    """4096 x 32768 Laplace activations with outliers, subnormals, NaN and Inf; k in {2, 4, 8}."""
    x, scale = workloads.fp8_activations(fmt, device="cuda")
    n = x.numel()
    slices = _slices(n, 8192, 8, 4)
    # make sure the special values are inside what the oracle sees
    special = torch.nonzero(~torch.isfinite(x)).flatten()[:64].cpu().numpy()
    slices += [(max(0, int(s) - 100), min(n, int(s) + 100)) for s in special[:8]]
    xs = [x[a:b].cpu().numpy() for a, b in slices]
    for k in (2, 4, 8):
        for variant in VARIANTS:
            out = fbsr.fbsr_round(x, fmt, variant, k, seed=7, scale=scale)
            for (a, b), xh in zip(slices, xs):
                gu.assert_codes_equal(out[a:b], capi.fbsr_round(xh, fmt, variant, k, seed=7, offset=a, scale=scale),
                                      "%s %s k=%d slice %d" % (fmt, variant, k, a))
    # whole-tensor counts of the special paths
    codes = fbsr.fbsr_round(x, fmt, "srf", 4, seed=7, scale=scale)
    mag = codes & 0x7F
    nan_code, max_code = 0x7F, (0x7E if fmt == "e4m3" else 0x7B)
    assert int((mag == nan_code).sum()) == 64
    assert int((mag == max_code).sum()) >= 2000
    if fmt == "e5m2":
        assert int((mag == 0x7C).sum()) == 128


def test_fused_optimizer_full_size():
    """The 32-block parameter list (1 979 711 488 fp32 parameters), SGD-momentum and Adam, 10 steps with
    step-indexed seeds; master weights, moments and bf16 codes checked on slices after steps 1 and 10."""
    n = workloads.optimizer_param_count(32)
    slices = _slices(n, 4096, 6, 5)
    for algo in ("sgd", "adam"):
        w, m, v = workloads.optimizer_state(n, device="cuda")
        g = torch.empty(n, dtype=torch.float32, device="cuda")
        lp = torch.empty(n, dtype=torch.uint16, device="cuda")
        host = [[t[a:b].cpu().numpy().copy() for t in (w, m, v)] for a, b in slices]
        for step in range(1, 11):
            workloads.optimizer_grad(n, step, device="cuda", out=g)
            k = (2, 4, 8)[step % 3]
            if algo == "sgd":
                fbsr.fbsr_sgd_update(w, g, m, "bf16", "srf", k, seed=50 + step, offset=0, lr=1e-4, mu=0.9, out=lp)
            else:
                fbsr.fbsr_adam_update(w, g, m, v, "bf16", "src", k, seed=50 + step, offset=0, lr=1e-4, beta1=0.9,
                                      beta2=0.999, eps=1e-8, step=step, out=lp)
            for (a, b), (wh, mh, vh) in zip(slices, host):
                gh = g[a:b].cpu().numpy()
                if algo == "sgd":
                    e = capi.sgd_update(wh, gh, mh, "bf16", "srf", k, seed=50 + step, offset=a, lr=1e-4, mu=0.9)
                else:
                    e = capi.adam_update(wh, gh, mh, vh, "bf16", "src", k, seed=50 + step, offset=a, lr=1e-4, beta1=0.9,
                                         beta2=0.999, eps=1e-8, step=step)
                if step in (1, 10):
                    gu.assert_codes_equal(lp[a:b], e, "%s step %d slice %d" % (algo, step, a))
                    assert np.array_equal(w[a:b].cpu().numpy().view(np.uint32), wh.view(np.uint32))
                    assert np.array_equal(m[a:b].cpu().numpy().view(np.uint32), mh.view(np.uint32))
                    if algo == "adam":
                        assert np.array_equal(v[a:b].cpu().numpy().view(np.uint32), vh.view(np.uint32))
        del w, m, v, g, lp
        torch.cuda.empty_cache()


def test_small_update_accumulation_full_size():
    """2^24 bfloat16 weights, 60 steps of updates of at most 2^-12 ulp: steps 1, 2 and 60 are checked against
    the oracle applied to the GPU's previous state; drift of mean |w| against exact fp64 accumulation."""
    n = 1 << 24
    w0 = workloads.accumulation_weights(n, device="cuda")
    for k, variant in ((1, "srff"), (2, "srf"), (4, "src"), (4, "srff")):
        w = w0.clone()
        exact = w0.view(torch.bfloat16).double()
        for step in range(1, 61):
            u = workloads.accumulation_update(w, step)
            exact += u.double()
            before = gu.to_np(w).copy() if step in (1, 2, 60) else None
            fbsr.fbsr_accumulate(w, u, "bf16", variant, k, seed=step, offset=0)
            if before is not None:
                expect = capi.accumulate(before, u.cpu().numpy(), "bf16", variant, k, seed=step, offset=0)
                gu.assert_codes_equal(w, expect, "%s k=%d step %d" % (variant, k, step))
        drift = (w.view(torch.bfloat16).double().abs().mean() - exact.abs().mean()).item()
        scale = w0.view(torch.bfloat16).double().abs().mean().item()
        if variant == "srff":
            assert drift < -1e-4 * scale * 2.0 ** -k        # systematic shrink of |w| (bias toward zero)
        else:
            assert abs(drift) < 1e-6 * scale                # weights do not move; only the tiny exact sum differs
