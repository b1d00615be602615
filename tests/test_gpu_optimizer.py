"""GPU parity for the fused SGD-momentum / Adam updates and low-precision accumulation."""
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


def _state(n, seed):
    w, m, v = workloads.optimizer_state(n, seed=seed, device="cuda")
    return w, m, v


@pytest.mark.parametrize("fmt", FMTS)
def test_sgd_momentum_steps(fmt):
    """Three consecutive steps with step-indexed seeds; master weights, momentum and codes bit-exact."""
    for k, variant in ((2, "srff"), (3, "src"), (4, "srf"), (8, "src"), (16, "srf")):
        n = 7 * fbsr.fbsr_tile_elements(k) + 19
        w, m, _ = _state(n, 40 + k)
        wh, mh = w.cpu().numpy().copy(), m.cpu().numpy().copy()
        for step in (1, 2, 3):
            g = workloads.optimizer_grad(n, step, device="cuda")
            out = fbsr.fbsr_sgd_update(w, g, m, fmt, variant, k, seed=500 + step, offset=0, lr=1e-4, mu=0.9)
            ecodes = capi.sgd_update(wh, g.cpu().numpy(), mh, fmt, variant, k, seed=500 + step, offset=0, lr=1e-4, mu=0.9)
            torch.cuda.synchronize()
            assert np.array_equal(w.cpu().numpy().view(np.uint32), wh.view(np.uint32))
            assert np.array_equal(m.cpu().numpy().view(np.uint32), mh.view(np.uint32))
            gu.assert_codes_equal(out, ecodes, "sgd %s k=%d step %d" % (fmt, k, step))


@pytest.mark.parametrize("fmt", ["bf16", "e4m3"])
def test_adam_steps(fmt):
    for k, variant in ((2, "srf"), (4, "src"), (6, "srff"), (8, "srf"), (13, "src")):
        n = 5 * fbsr.fbsr_tile_elements(k) + 3
        w, m, v = _state(n, 60 + k)
        wh, mh, vh = (t.cpu().numpy().copy() for t in (w, m, v))
        for step in (1, 2, 3, 10):
            g = workloads.optimizer_grad(n, step, device="cuda")
            out = fbsr.fbsr_adam_update(w, g, m, v, fmt, variant, k, seed=900 + step, offset=0, lr=1e-4,
                                        beta1=0.9, beta2=0.999, eps=1e-8, step=step)
            ecodes = capi.adam_update(wh, g.cpu().numpy(), mh, vh, fmt, variant, k, seed=900 + step, offset=0,
                                      lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, step=step)
            torch.cuda.synchronize()
            for got, exp, name in ((w, wh, "w"), (m, mh, "m"), (v, vh, "v")):
                assert np.array_equal(got.cpu().numpy().view(np.uint32), exp.view(np.uint32)), name
            gu.assert_codes_equal(out, ecodes, "adam %s k=%d step %d" % (fmt, k, step))


def test_optimizer_unaligned_and_offset():
    n = 20_011
    w, m, v = _state(n + 4, 70)
    g = workloads.optimizer_grad(n + 4, 1, device="cuda")
    wh, mh, vh, gh = (t.cpu().numpy().copy() for t in (w, m, v, g))
    out = fbsr.fbsr_adam_update(w[1:n + 1], g[3:n + 3], m[2:n + 2], v[:n], "bf16", "srf", 4, seed=1, offset=12345,
                                lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=4)
    w1, m1, v1 = wh[1:n + 1].copy(), mh[2:n + 2].copy(), vh[:n].copy()
    e = capi.adam_update(w1, gh[3:n + 3], m1, v1, "bf16", "srf", 4, seed=1, offset=12345, lr=1e-3, beta1=0.9,
                         beta2=0.999, eps=1e-8, step=4)
    torch.cuda.synchronize()
    assert np.array_equal(w.cpu().numpy()[1:n + 1].view(np.uint32), w1.view(np.uint32))
    assert w.cpu().numpy()[0] == wh[0] and np.array_equal(w.cpu().numpy()[n + 1:], wh[n + 1:])
    gu.assert_codes_equal(out, e, "adam unaligned")


@pytest.mark.parametrize("fmt", FMTS)
def test_accumulate(fmt):
    rng = np.random.default_rng(81)
    for k, variant in ((1, "srff"), (2, "srf"), (4, "src"), (5, "srf"), (11, "srff")):
        n = 6 * fbsr.fbsr_tile_elements(k) + 21
        bits = 16 if fmt in ("bf16", "fp16") else 8
        codes = rng.integers(0, 1 << bits, size=n).astype(capi.CODE_DTYPE[fmt])      # every code, NaN/Inf included
        vals = capi.decode_array(fmt, codes)
        u = (np.nan_to_num(vals, nan=1.0, posinf=1.0, neginf=-1.0) * rng.uniform(-0.05, 0.05, n)).astype(np.float32)
        wd = gu.from_np_codes(codes)
        fbsr.fbsr_accumulate(wd, torch.from_numpy(u).cuda(), fmt, variant, k, seed=21, offset=2)
        expect = capi.accumulate(codes.copy(), u, fmt, variant, k, seed=21, offset=2)
        gu.assert_codes_equal(wd, expect, "accumulate %s k=%d" % (fmt, k))


def test_small_update_accumulation_drift():
    """Config 'small-update accumulation' at 2^18 weights and 20 steps: each step is checked against
    the oracle applied to the GPU's previous state; SRF/SRC never move a weight, SRFF drifts toward zero."""
    n = 1 << 18
    w0 = workloads.accumulation_weights(n, device="cuda")
    for k in (1, 2, 4):
        for variant in VARIANTS:
            w = w0.clone()
            for step in range(1, 21):
                u = workloads.accumulation_update(w, step)
                before = gu.to_np(w).copy()
                fbsr.fbsr_accumulate(w, u, "bf16", variant, k, seed=step, offset=0)
                if step in (1, 2, 20):
                    expect = capi.accumulate(before, u.cpu().numpy(), "bf16", variant, k, seed=step, offset=0)
                    gu.assert_codes_equal(w, expect, "accum %s k=%d step %d" % (variant, k, step))
            moved = (w != w0).float().mean().item()
            if variant == "srff":
                assert 0.3 * (1 - (1 - 2.0 ** -k / 2) ** 20) < moved <= 1.0
                drift = (w.view(torch.bfloat16).float().abs().double().mean()
                         - w0.view(torch.bfloat16).float().abs().double().mean()).item()
                assert drift < 0
            else:
                assert moved == 0.0
