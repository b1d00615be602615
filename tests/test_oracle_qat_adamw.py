"""Pins for the oracle's whole Algorithm-1 iteration (gradient -> AdamW update in F16 -> RoundTo8 with SR).

The paper fixes the shape of the step (Algorithm 1) but not its arithmetic, so the operation list is the library's
own; it is pinned by: exact-rational replay of every operation (tier 0 against tier 1), Adam's first-step closed
form (the update is -lr sign(g)), torch.optim.AdamW run on the widened weights, and the separately pinned
16-bit-sum rounding step (fbsr qat_update), which the tail of the fused step must equal.
"""
import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import VARIANTS, f32_bits

W_FMTS = ("e4m3", "e5m2", "b8p4")
G_DTYPE = {"bf16": torch.bfloat16, "fp16": torch.float16}


def finite_weight_codes(rng, fmt, n):
    codes = rng.integers(0, 256, size=n).astype(np.uint8)
    vals = capi.decode_array(fmt, codes)
    codes[~np.isfinite(vals)] = 0x38
    return codes


def to16(x, g_fmt):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(G_DTYPE[g_fmt]).view(torch.int16).numpy().view(np.uint16).copy()


@pytest.mark.parametrize("w_fmt", W_FMTS)
@pytest.mark.parametrize("g_fmt", ["bf16", "fp16"])
def test_exact_rational_replay(w_fmt, g_fmt):
    rng = np.random.default_rng(51)
    n = 160
    w8 = finite_weight_codes(rng, w_fmt, n)
    g16 = to16(rng.standard_normal(n) * 10.0 ** rng.uniform(-4, 0, n), g_fmt)
    g16[:4] = [0x0000, 0x8000, 0x0001, 0x8001]                                  # zeros and the smallest subnormals
    m = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    v = (rng.uniform(0, 1e-3, n)).astype(np.float32)
    lr, b1, b2, eps, wd, step = np.float32(3e-3), np.float32(0.9), np.float32(0.95), np.float32(1e-8), np.float32(0.1), 3
    for variant, k in (("srff", 3), ("srf", 3), ("src", 3), ("rtne", 1), ("src", 9)):
        w1, m1, v1 = w8.copy(), m.copy(), v.copy()
        capi.qat_adamw_step(w1, g16, m1, v1, w_fmt, g_fmt, variant, k, seed=7, offset=40, lr=float(lr), beta1=float(b1),
                            beta2=float(b2), eps=float(eps), weight_decay=float(wd), step=step)
        c1, c2, a1, a2 = pl.adam_coefficients(int(f32_bits(lr)), int(f32_bits(b1)), int(f32_bits(b2)), step)
        lrwd = int(f32_bits(np.float32(lr * wd)))
        for i in range(n):
            nr = capi.draw(7, 40 + i, k)
            code, m2, v2, _ = pl.qat_adamw_step(int(w8[i]), int(g16[i]), int(f32_bits(m[i])), int(f32_bits(v[i])), w_fmt, g_fmt,
                                                variant, nr, k, int(f32_bits(b1)), int(f32_bits(b2)), int(f32_bits(eps)),
                                                c1, c2, a1, a2, lrwd)
            assert code == int(w1[i]) and m2 == int(f32_bits(m1[i])) and v2 == int(f32_bits(v1[i])), (variant, i)


@pytest.mark.parametrize("g_fmt", ["bf16", "fp16"])
def test_first_step_is_minus_lr_sign_g(g_fmt):
    """Step 1 from zero moments, no decay: c1 m' = lr g and sqrt(v') c2 = |g|, so u = -lr g / (|g| + eps) = -lr sign(g)
    up to a few binary32 roundings; with lr a power of two u16 is exactly -+lr, and the weight moves by that."""
    rng = np.random.default_rng(53)
    n = 400
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-3, 1, n)).astype(np.float32)
    g16 = to16(g, g_fmt)
    gv = capi.decode_array(g_fmt, g16)
    lr = 2.0 ** -7
    c1, c2, a1, a2 = pl.adam_coefficients(int(f32_bits(np.float32(lr))), int(f32_bits(np.float32(0.9))),
                                          int(f32_bits(np.float32(0.999))), 1)
    for i in range(0, n, 7):
        _, _, _, u16 = pl.qat_adamw_step(0x38, int(g16[i]), 0, 0, "e4m3", g_fmt, "srf", 0, 3, int(f32_bits(np.float32(0.9))),
                                         int(f32_bits(np.float32(0.999))), int(f32_bits(np.float32(1e-12))), c1, c2, a1, a2, 0)
        assert capi.decode(g_fmt, u16) == -lr * np.sign(gv[i])
    # weights on the grid of spacing 2^-6 >= lr: with all excess bits drawn (k = 4 >= D) SR moves each weight to a
    # neighbour, down for g > 0 and up for g < 0, or leaves it
    w8 = np.full(n, 0x30, dtype=np.uint8)                                   # 0.5 in E4M3, ulp 2^-4
    w1, m, v = w8.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    capi.qat_adamw_step(w1, g16, m, v, "e4m3", g_fmt, "srf", 5, seed=1, offset=0, lr=lr, beta1=0.9, beta2=0.999, eps=1e-12,
                        weight_decay=0.0, step=1)
    moved = capi.decode_array("e4m3", w1) - 0.5
    assert np.all((moved == 0) | (np.sign(moved) == -np.sign(gv)))
    # exact SR of a step of 1/8 ulp below a binade boundary (ulp 2^-5 below 0.5): P(up) = 1/4 for g > 0 ...
    frac = np.mean(moved[gv > 0] != 0)
    assert 0.12 < frac < 0.40


@pytest.mark.parametrize("w_fmt", W_FMTS)
def test_update_matches_torch_adamw(w_fmt):
    """u = w_new - w of torch.optim.AdamW on the widened weights, to binary32 accuracy: the u16 of the oracle is within
    one F16 ulp of torch's update rounded to F16 (a different but equivalent operation order)."""
    rng = np.random.default_rng(57)
    n = 500
    w8 = finite_weight_codes(rng, w_fmt, n)
    wv = capi.decode_array(w_fmt, w8).astype(np.float32)
    lr, b1, b2, eps, wd = 1e-2, 0.9, 0.95, 1e-8, 0.1
    p = torch.nn.Parameter(torch.from_numpy(wv.copy()))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    for step in (1, 2, 3):
        g = (rng.standard_normal(n) * 0.1).astype(np.float32)
        g16 = to16(g, "bf16")
        gv = capi.decode_array("bf16", g16).astype(np.float32)
        before = p.detach().numpy().copy()
        p.grad = torch.from_numpy(gv.copy())
        opt.step()
        u_torch = p.detach().numpy().astype(np.float64) - before
        # our update for the same weights and moments: replay tier 0 to get u16
        c1, c2, a1, a2 = pl.adam_coefficients(int(f32_bits(np.float32(lr))), int(f32_bits(np.float32(b1))),
                                              int(f32_bits(np.float32(b2))), step)
        # the oracle's moments track torch's (same recurrences) to binary32 accuracy
        m1, v1 = m.copy(), v.copy()
        w1 = w8.copy()
        capi.qat_adamw_step(w1, g16, m1, v1, w_fmt, "bf16", "rtne", 1, seed=0, offset=0, lr=lr, beta1=b1, beta2=b2, eps=eps,
                            weight_decay=wd, step=step)
        st = opt.state[p]
        assert np.allclose(m1, st["exp_avg"].numpy(), rtol=1e-5, atol=1e-8)       # atol: the two terms can cancel
        assert np.allclose(v1, st["exp_avg_sq"].numpy(), rtol=1e-5, atol=1e-12)
        if step == 1:
            for i in range(0, n, 5):
                _, _, _, u16 = pl.qat_adamw_step(int(w8[i]), int(g16[i]), 0, 0, w_fmt, "bf16", "rtne", 0, 1,
                                                 int(f32_bits(np.float32(b1))), int(f32_bits(np.float32(b2))),
                                                 int(f32_bits(np.float32(eps))), c1, c2, a1, a2,
                                                 int(f32_bits(np.float32(np.float32(lr) * np.float32(wd)))))
                ours = capi.decode("bf16", u16)
                ulp16 = 2.0 ** (np.floor(np.log2(abs(u_torch[i]) + 1e-30)) - 7)
                assert abs(ours - u_torch[i]) <= ulp16 * 0.51 + abs(wv[i]) * 2e-7, i
        m, v = m1, v1
        # torch keeps its own weights: feed it the same ones next step
        with torch.no_grad():
            p.copy_(torch.from_numpy(wv))


@pytest.mark.parametrize("w_fmt", W_FMTS)
@pytest.mark.parametrize("variant", VARIANTS)
def test_tail_equals_the_16_bit_sum_step(w_fmt, variant):
    """The fused step = (u16 from the update) followed by the separately pinned w8 <- RoundTo8(w16 + u16)."""
    rng = np.random.default_rng(59)
    n = 300
    w8 = finite_weight_codes(rng, w_fmt, n)
    g16 = to16(rng.standard_normal(n) * 0.3, "fp16")
    m = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    v = rng.uniform(1e-6, 1e-2, n).astype(np.float32)
    lr, b1, b2, eps, wd, step = np.float32(0.05), np.float32(0.9), np.float32(0.999), np.float32(1e-8), np.float32(0.01), 5
    c1, c2, a1, a2 = pl.adam_coefficients(int(f32_bits(lr)), int(f32_bits(b1)), int(f32_bits(b2)), step)
    u16 = np.array([pl.qat_adamw_step(int(w8[i]), int(g16[i]), int(f32_bits(m[i])), int(f32_bits(v[i])), w_fmt, "fp16", variant, 0, 3,
                                      int(f32_bits(b1)), int(f32_bits(b2)), int(f32_bits(eps)), c1, c2, a1, a2,
                                      int(f32_bits(np.float32(lr * wd))))[3] for i in range(n)], dtype=np.uint16)
    two_calls = capi.qat_update(w8.copy(), u16, w_fmt, "fp16", variant, 3, seed=9, offset=2)
    fused = w8.copy()
    capi.qat_adamw_step(fused, g16, m.copy(), v.copy(), w_fmt, "fp16", variant, 3, seed=9, offset=2, lr=float(lr), beta1=float(b1),
                        beta2=float(b2), eps=float(eps), weight_decay=float(wd), step=step)
    assert np.array_equal(fused, two_calls)


def test_zero_gradient_and_no_decay_leave_the_weights():
    rng = np.random.default_rng(61)
    w8 = finite_weight_codes(rng, "b8p4", 512)
    g16 = np.zeros(512, dtype=np.uint16)
    for variant in VARIANTS + ("rtne",):
        w1 = w8.copy()
        m, v = np.zeros(512, np.float32), np.zeros(512, np.float32)
        capi.qat_adamw_step(w1, g16, m, v, "b8p4", "bf16", variant, 3, seed=3, offset=0, lr=1e-2, beta1=0.9, beta2=0.999,
                            eps=1e-8, weight_decay=0.0, step=1)
        expect = w8.copy()
        expect[expect == 0x80] = 0x00
        assert np.array_equal(w1, expect) and not m.any() and not v.any()
