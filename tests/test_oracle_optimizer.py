"""Pins for the fused-update steps of the oracle (last line of Algorithm 1: the new weight is
computed in the wide format, then SR-rounded).  The binary32 operation list is this library's
own definition, so it is pinned by: exact-rational evaluation with one rounding per operation
(tier 0), torch's SGD/Adam as a loose sanity reference, and composition with the rounding
oracle that the other test modules pin."""
import numpy as np
import pytest
import torch

from oracle import capi, paper_literal as pl
from helpers import bits_f32, f32_bits, random_f32, VARIANTS


def test_sgd_momentum_against_exact_arithmetic_and_torch():
    rng = np.random.default_rng(31)
    n = 300
    w = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    m = rng.normal(0, 1e-3, n).astype(np.float32)
    lr, mu = np.float32(1e-4), np.float32(0.9)
    w1, m1 = w.copy(), m.copy()
    codes = capi.sgd_update(w1, g, m1, "bf16", "srf", 4, seed=3, offset=10, lr=float(lr), mu=float(mu))
    for i in range(n):
        w2, m2 = pl.sgd_momentum_step(int(f32_bits(w[i])), int(f32_bits(g[i])), int(f32_bits(m[i])),
                                      int(f32_bits(lr)), int(f32_bits(mu)))
        assert w2 == int(f32_bits(w1[i])) and m2 == int(f32_bits(m1[i]))
    # the low-precision output is the rounding oracle applied to the new master weight
    assert np.array_equal(codes, capi.fbsr_round(w1, "bf16", "srf", 4, seed=3, offset=10))
    # torch.optim.SGD computes the same recurrence (different rounding order): a few ulps
    p = torch.nn.Parameter(torch.from_numpy(w.copy()))
    opt = torch.optim.SGD([p], lr=float(lr), momentum=float(mu))
    opt.state[p]["momentum_buffer"] = torch.from_numpy(m.copy())
    p.grad = torch.from_numpy(g.copy())
    opt.step()
    assert np.allclose(p.detach().numpy(), w1, rtol=1e-6, atol=1e-9)
    assert np.allclose(opt.state[p]["momentum_buffer"].numpy(), m1, rtol=1e-6, atol=1e-9)


@pytest.mark.parametrize("step", [1, 2, 10])
def test_adam_against_exact_arithmetic_and_torch(step):
    rng = np.random.default_rng(32 + step)
    n = 200
    w = rng.normal(0, 0.02, n).astype(np.float32)
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    m = (rng.normal(0, 1e-4, n) * (step > 1)).astype(np.float32)
    v = (rng.uniform(0, 1e-7, n) * (step > 1)).astype(np.float32)
    lr, b1, b2, eps = np.float32(1e-4), np.float32(0.9), np.float32(0.999), np.float32(1e-8)
    w1, m1, v1 = w.copy(), m.copy(), v.copy()
    codes = capi.adam_update(w1, g, m1, v1, "bf16", "src", 8, seed=5, offset=0, lr=float(lr),
                             beta1=float(b1), beta2=float(b2), eps=float(eps), step=step)
    c = capi.adam_coefficients(float(lr), float(b1), float(b2), step)
    c0 = pl.adam_coefficients(int(f32_bits(lr)), int(f32_bits(b1)), int(f32_bits(b2)), step)
    assert tuple(int(f32_bits(x)) for x in c) == c0
    for i in range(n):
        w2, m2, v2 = pl.adam_step(int(f32_bits(w[i])), int(f32_bits(g[i])), int(f32_bits(m[i])),
                                  int(f32_bits(v[i])), int(f32_bits(b1)), int(f32_bits(b2)),
                                  int(f32_bits(eps)), *c0)
        assert (w2, m2, v2) == (int(f32_bits(w1[i])), int(f32_bits(m1[i])), int(f32_bits(v1[i])))
    assert np.array_equal(codes, capi.fbsr_round(w1, "bf16", "src", 8, seed=5, offset=0))
    # torch.optim.Adam, same hyper-parameters and step count, loose tolerance
    p = torch.nn.Parameter(torch.from_numpy(w.copy()))
    opt = torch.optim.Adam([p], lr=float(lr), betas=(float(b1), float(b2)), eps=float(eps))
    opt.state[p]["step"] = torch.tensor(float(step - 1))
    opt.state[p]["exp_avg"] = torch.from_numpy(m.copy())
    opt.state[p]["exp_avg_sq"] = torch.from_numpy(v.copy())
    p.grad = torch.from_numpy(g.copy())
    opt.step()
    assert np.allclose(opt.state[p]["exp_avg"].numpy(), m1, rtol=1e-5, atol=1e-12)
    assert np.allclose(opt.state[p]["exp_avg_sq"].numpy(), v1, rtol=1e-5, atol=1e-15)
    assert np.allclose(p.detach().numpy(), w1, rtol=1e-5, atol=1e-8)


@pytest.mark.parametrize("fmt", ["bf16", "fp16", "e4m3", "e5m2"])
def test_accumulate_is_decode_add_round(fmt):
    rng = np.random.default_rng(33)
    n = 500
    w0 = rng.integers(0, 1 << (16 if fmt in ("bf16", "fp16") else 8), size=n).astype(capi.CODE_DTYPE[fmt])
    vals = capi.decode_array(fmt, w0)
    keep = np.isfinite(vals)
    w0, vals = w0[keep], vals[keep]
    u = (vals * rng.uniform(-0.01, 0.01, vals.size)).astype(np.float32)
    w = w0.copy()
    capi.accumulate(w, u, fmt, "srf", 3, seed=8, offset=2)
    y = (vals + u).astype(np.float32)
    assert np.array_equal(w, capi.fbsr_round(y, fmt, "srf", 3, seed=8, offset=2))


def test_small_updates_stagnate_or_drift_as_the_predicates_dictate():
    """Updates of at most 2^-12 target ulp with k <= 4 bits: delta is below 2^-12 (or above
    1 - 2^-12).  SRF and SRC then behave like round-to-nearest (no weight moves: the
    'stagnation' of Section IV), SRFF moves a weight one ulp toward zero with probability
    2^-k when the update points toward zero and never moves it otherwise."""
    rng = np.random.default_rng(34)
    n = 1 << 16
    w32 = rng.normal(0, 0.02, n).astype(np.float32)
    w0 = torch.from_numpy(w32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    vals = capi.decode_array("bf16", w0)
    ulp = np.ldexp(1.0, np.maximum(np.frexp(np.abs(vals))[1] - 1, -126) - 7)
    c = rng.uniform(0.05, 1.0, n)
    toward_zero = rng.integers(0, 2, n).astype(bool)
    u = (np.where(toward_zero, -1.0, 1.0) * np.sign(vals) * c * 2.0 ** -12 * ulp).astype(np.float32)
    for k in (1, 2, 4):
        for variant in ("srf", "src"):
            w = w0.copy()
            capi.accumulate(w, u, "bf16", variant, k, seed=1, offset=0)
            assert np.array_equal(w, w0)
        w = w0.copy()
        capi.accumulate(w, u, "bf16", "srff", k, seed=1, offset=0)
        moved = w != w0
        assert not moved[~toward_zero].any()
        frac = moved[toward_zero].mean()
        # draws with n = 0 keep the (truncated) value one ulp below: probability 2^-k
        assert abs(frac - 2.0 ** -k) < 5 * np.sqrt(2.0 ** -k / toward_zero.sum()) + 1e-3
        assert np.all(np.abs(capi.decode_array("bf16", w[moved])) < np.abs(vals[moved]))
