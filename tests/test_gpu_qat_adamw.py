"""GPU parity for fbsr_qat_adamw_step (one whole iteration of Algorithm 1, fused) against the oracle: weight codes
bit for bit, moments bit for bit where finite."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from helpers import VARIANTS  # noqa: E402

HYPER = dict(lr=3e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from oracle import capi
    import gpu_util
    module.fbsr, module.capi, module.gu = fbsr, capi, gpu_util


def make_case(rng, w_fmt, g_fmt, n, specials=True):
    w8 = rng.integers(0, 256, size=n).astype(np.uint8)
    vals = capi.decode_array(w_fmt, w8)
    if not specials:
        w8[~np.isfinite(vals)] = 0x38
    dt = torch.bfloat16 if g_fmt == "bf16" else torch.float16
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-5, 0, n)).astype(np.float32)
    g16 = torch.from_numpy(g).to(dt).view(torch.int16).numpy().view(np.uint16).copy()
    if specials:
        g16[rng.choice(n, size=24, replace=False)] = rng.integers(0, 1 << 16, size=24).astype(np.uint16)   # arbitrary codes, NaN / Inf among them
        g16[:4] = [0x0000, 0x8000, 0x0001, 0x8001]
    m = (rng.standard_normal(n) * 1e-2).astype(np.float32)
    v = rng.uniform(0, 1e-3, n).astype(np.float32)
    return w8, g16, m, v


def same_state(a_t, b_np):
    a = a_t.cpu().numpy()
    fin = np.isfinite(b_np)
    return np.array_equal(a.view(np.uint32)[fin], b_np.view(np.uint32)[fin]) and np.array_equal(np.isnan(a), np.isnan(b_np)) \
        and np.array_equal(a[~fin & ~np.isnan(b_np)], b_np[~fin & ~np.isnan(b_np)])


@pytest.mark.parametrize("w_fmt", ["e4m3", "e5m2", "b8p4"])
@pytest.mark.parametrize("g_fmt", ["bf16", "fp16"])
def test_parity_every_variant(w_fmt, g_fmt):
    rng = np.random.default_rng(71)
    for variant, k, step in (("srff", 3, 1), ("srf", 3, 2), ("src", 3, 7), ("rtne", 1, 3), ("src", 6, 1), ("srf", 10, 4),
                             ("srff", 16, 2), ("rta", 1, 1)):
        n = 7 * fbsr.fbsr_tile_elements(k) + 29
        w8, g16, m, v = make_case(rng, w_fmt, g_fmt, n)
        wd, gd = gu.from_np_codes(w8), gu.from_np_codes(g16)
        md, vd = torch.from_numpy(m).cuda(), torch.from_numpy(v).cuda()
        fbsr.fbsr_qat_adamw_step(wd, gd, md, vd, w_fmt, g_fmt, variant, k, seed=11, offset=6, step=step, **HYPER)
        w1, m1, v1 = w8.copy(), m.copy(), v.copy()
        capi.qat_adamw_step(w1, g16, m1, v1, w_fmt, g_fmt, variant, k, seed=11, offset=6, step=step, **HYPER)
        gu.assert_codes_equal(wd, w1, "%s<-%s %s k=%d" % (w_fmt, g_fmt, variant, k))
        assert same_state(md, m1) and same_state(vd, v1)


def test_updates_beyond_the_16_bit_range_saturate():
    """A learning rate so large that the update overflows binary16: u16 saturates at -+65504 (it does not become an
    infinity), and so does the 16-bit sum."""
    rng = np.random.default_rng(79)
    for w_fmt in ("e5m2", "b8p4", "e4m3"):
        n = 6 * 1536 + 11
        w8, g16, m, v = make_case(rng, w_fmt, "fp16", n, specials=False)
        for lr in (1e6, 3e4):
            wd, gd = gu.from_np_codes(w8), gu.from_np_codes(g16)
            md, vd = torch.from_numpy(m).cuda(), torch.from_numpy(v).cuda()
            kw = dict(lr=lr, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
            fbsr.fbsr_qat_adamw_step(wd, gd, md, vd, w_fmt, "fp16", "srf", 5, seed=1, offset=0, step=1, **kw)
            w1, m1, v1 = w8.copy(), m.copy(), v.copy()
            capi.qat_adamw_step(w1, g16, m1, v1, w_fmt, "fp16", "srf", 5, seed=1, offset=0, step=1, **kw)
            gu.assert_codes_equal(wd, w1, "%s lr=%g" % (w_fmt, lr))
            assert same_state(md, m1) and same_state(vd, v1)
            # most weights end at the largest finite value, none at an infinity
            top8 = {"e5m2": 0x7B, "b8p4": 0x7E, "e4m3": 0x7E}[w_fmt]
            assert not np.any((w1 & 0x7F) == 0x7F) and (lr < 1e6 or np.mean((w1 & 0x7F) == top8) > 0.5)


def test_unaligned_pointers_offsets_and_small_sizes():
    rng = np.random.default_rng(73)
    for n in (0, 1, 7, 255, 3000):
        for skip in (0, 1, 3):
            for offset in (0, 5, 2 ** 40 + 1):
                w8, g16, m, v = make_case(rng, "b8p4", "bf16", n + 8, specials=False)
                wd, gd = gu.from_np_codes(w8), gu.from_np_codes(g16)
                md, vd = torch.from_numpy(m).cuda(), torch.from_numpy(v).cuda()
                fbsr.fbsr_qat_adamw_step(wd[skip:skip + n], gd[skip:skip + n], md[skip:skip + n], vd[skip:skip + n], "b8p4", "bf16",
                                         "src", 3, seed=2, offset=offset, step=2, **HYPER)
                w1, m1, v1 = w8.copy(), m.copy(), v.copy()
                capi.qat_adamw_step(w1[skip:skip + n], g16[skip:skip + n], m1[skip:skip + n], v1[skip:skip + n], "b8p4", "bf16", "src", 3,
                                    seed=2, offset=offset, step=2, **HYPER)
                gu.assert_codes_equal(wd, w1, "n=%d skip=%d offset=%d" % (n, skip, offset))       # untouched neighbours included
                assert same_state(md, m1) and same_state(vd, v1)


def test_equals_update_then_rounding_step():
    """The fused call equals torch-side composition of the library's own pieces: no piece alone, but u16 recovered
    from a zero weight decay, zero-moment first step is -lr sign(g), so w8 must equal fbsr_qat_update with that u16."""
    n = 1 << 20
    g = torch.Generator(device="cuda").manual_seed(3)
    w8 = fbsr.fbsr_round(torch.rand(n, device="cuda", generator=g) + 0.5, "b8p4", "rtne", 1, seed=0)
    grad = torch.randn(n, device="cuda", generator=g)
    g16 = grad.to(torch.bfloat16).view(torch.uint16)
    lr = 2.0 ** -7
    u16 = (-lr * torch.sign(grad.to(torch.bfloat16).float())).to(torch.bfloat16).view(torch.uint16)
    for variant in VARIANTS:
        a = w8.clone()
        fbsr.fbsr_qat_adamw_step(a, g16, torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda"), "b8p4", "bf16", variant, 3,
                                 seed=5, offset=0, lr=lr, beta1=0.9, beta2=0.999, eps=1e-12, weight_decay=0.0, step=1)
        b = w8.clone()
        fbsr.fbsr_qat_update(b, u16, "b8p4", "bf16", variant, 3, seed=5, offset=0)
        assert torch.equal(a, b)


def test_training_loop_in_miniature():
    """Section IV's observation on a quadratic: minimise sum (w - target)^2 / 2 over Binary8P4 weights with BFloat16
    gradients and 3 random bits.  Round-to-nearest stagnates once the update falls under half an ulp; SRC and SRF keep
    descending; every step is checked against the oracle on a slice."""
    n = 1 << 18
    g = torch.Generator(device="cuda").manual_seed(9)
    target = torch.rand(n, device="cuda", generator=g) * 0.5 + 1.0           # [1, 1.5), ulp 1/8
    w0 = fbsr.fbsr_round(torch.full((n,), 1.75, device="cuda"), "b8p4", "rtne", 1, seed=0)
    table = torch.from_numpy(capi.decode_array("b8p4", np.arange(256, dtype=np.uint8)).astype(np.float32)).cuda()
    loss = {}
    for variant in ("rtne", "srff", "srf", "src"):
        w = w0.clone()
        m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        for step in range(1, 41):
            grad16 = (table[w.long()] - target).to(torch.bfloat16).view(torch.uint16)
            if step in (1, 17, 40):
                wb, mb, vb = gu.to_np(w)[:30000].copy(), m[:30000].cpu().numpy(), v[:30000].cpu().numpy()
                capi.qat_adamw_step(wb, gu.to_np(grad16)[:30000], mb, vb, "b8p4", "bf16", variant, 3, seed=step, offset=0,
                                    lr=2.0 ** -5, beta1=0.9, beta2=0.99, eps=1e-8, weight_decay=0.0, step=step)
            fbsr.fbsr_qat_adamw_step(w, grad16, m, v, "b8p4", "bf16", variant, 3, seed=step, offset=0,
                                     lr=2.0 ** -5, beta1=0.9, beta2=0.99, eps=1e-8, weight_decay=0.0, step=step)
            if step in (1, 17, 40):
                assert np.array_equal(gu.to_np(w)[:30000], wb) and same_state(m[:30000], mb) and same_state(v[:30000], vb)
        loss[variant] = float(((table[w.long()] - target) ** 2).mean()) / 2
    start = float(((table[w0.long()] - target) ** 2).mean()) / 2
    assert loss["rtne"] == start                        # updates of 1/4 ulp (lr = 2^-5, ulp 1/8): nearest never moves
    assert loss["src"] < 0.8 * start and loss["srf"] < 0.8 * start


def test_full_size_launch():
    n = (1 << 27) + 5
    g = torch.Generator(device="cuda").manual_seed(21)
    w = fbsr.fbsr_round(torch.randn(n, device="cuda", generator=g), "e4m3", "rtne", 1, seed=0)
    g16 = (torch.randn(n, device="cuda", generator=g) * 1e-2).to(torch.bfloat16).view(torch.uint16)
    m = torch.randn(n, device="cuda", generator=g) * 1e-3
    v = torch.rand(n, device="cuda", generator=g) * 1e-4
    w0, m0, v0 = w.clone(), m.clone(), v.clone()
    fbsr.fbsr_qat_adamw_step(w, g16, m, v, "e4m3", "bf16", "src", 3, seed=8, offset=0, step=3, **HYPER)
    for a in (0, 1280 * 40000, n - 4001):
        b = min(a + 4001, n)
        wb, mb, vb = gu.to_np(w0[a:b]).copy(), m0[a:b].cpu().numpy(), v0[a:b].cpu().numpy()
        capi.qat_adamw_step(wb, gu.to_np(g16[a:b]), mb, vb, "e4m3", "bf16", "src", 3, seed=8, offset=a, step=3, **HYPER)
        assert np.array_equal(gu.to_np(w[a:b]), wb) and same_state(m[a:b], mb) and same_state(v[a:b], vb)


def test_argument_errors():
    w = torch.zeros(64, dtype=torch.uint8, device="cuda")
    g16 = torch.zeros(64, dtype=torch.uint16, device="cuda")
    m, v = torch.zeros(64, device="cuda"), torch.zeros(64, device="cuda")
    with pytest.raises(fbsr.FbsrError) as err:
        fbsr.fbsr_qat_adamw_step(w, g16, m, v, "e4m3", "bf16", "src", 3, seed=0, offset=0, step=0, **HYPER)
    assert err.value.status == 1
    with pytest.raises(fbsr.FbsrError) as err:
        fbsr.fbsr_qat_adamw_step(w, g16, m, v, "e4m3", "e5m2", "src", 3, seed=0, offset=0, step=1, **HYPER)
    assert err.value.status == 2
