"""Whole-tensor parity, at the sizes the benchmark times, for the entry points beyond plain rounding: 16-bit
sources, block scales, supplied bits, run-time formats, Binary8P4 and the two Algorithm-1 steps.  As in
test_gpu_fullsize.py the oracle checks every element on all host cores; a cut would be printed and raised as a
warning."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def setup_module(module):
    import paper_2504_20634_b200 as fbsr
    from paper_2504_20634_b200 import workloads
    from oracle import capi
    import gpu_util
    capi.lib()
    module.fbsr, module.capi, module.gu, module.workloads = fbsr, capi, gpu_util, workloads


def _whole(n, what, pieces_fn, budget=90, calls=1, chk=None):
    own = chk is None
    chk = chk or gu.WholeTensorChecker(budget_s=budget)
    chk.run(n, pieces_fn, remaining_calls=calls)
    if own:
        chk.report(what)
        assert chk.fraction > 0.2
    return chk


def test_16_bit_sources_full_size():
    """2^28 BFloat16 codes to the three 8-bit formats, k = 3 (Section IV's setting), every variant."""
    n = 1 << 28
    codes = workloads.lp_sweep(n, "bf16", device="cuda")
    c_pin, ch = gu.pinned_like(codes)
    c_pin.copy_(codes)
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    o_pin, oh = gu.pinned_like(out)
    combos = [(f, v, s) for f in ("e4m3", "e5m2", "b8p4") for v in ("srff", "srf", "src") for s in (1.0,)] + [("e4m3", "src", 0.7)]
    chk = gu.WholeTensorChecker(budget_s=150)
    for idx, (dst_fmt, variant, scale) in enumerate(combos):
        fbsr.fbsr_round_lp(codes, "bf16", dst_fmt, variant, 3, seed=5, scale=scale, out=out)
        o_pin.copy_(out)
        torch.cuda.synchronize()
        _whole(n, "", lambda a, b: gu.first_difference(
            oh[a:b], capi.fbsr_round_lp(ch[a:b], "bf16", dst_fmt, variant, 3, seed=5, offset=a, scale=scale), a,
            "bf16->%s %s scale %g" % (dst_fmt, variant, scale)), calls=len(combos) - idx, chk=chk)
    chk.report("16-bit sources, 10 x 2^28")
    assert chk.fraction > 0.2


@pytest.mark.parametrize("fmt", ["e4m3", "bf16"])
def test_block_scales_full_size(fmt):
    n = 1 << 27
    x = workloads.bandwidth_sweep(n, seed=1234, device="cuda")
    out, sc = fbsr.fbsr_round_mx(x, fmt, "src", 3, seed=5)
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    o_pin, oh = gu.pinned_like(out)
    o_pin.copy_(out)
    s_pin, sh = gu.pinned_like(sc)
    s_pin.copy_(sc)
    torch.cuda.synchronize()

    def piece(a, b):
        ecodes, escales = capi.fbsr_round_mx(xh[a:b], fmt, "src", 3, seed=5, offset=a)
        return gu.first_difference(oh[a:b], ecodes, a, "block-scaled codes") or \
            gu.first_difference(sh[a // 32:(b + 31) // 32], escales, a // 32, "block scales")

    _whole(n, "block scales %s, 2^27" % fmt, piece)


def test_supplied_bits_full_size():
    n = 1 << 27
    x = workloads.bandwidth_sweep(n, seed=1234, device="cuda")
    k, dpw = 3, 10
    words = torch.randint(0, 2 ** 31, ((n + dpw - 1) // dpw,), device="cuda", dtype=torch.int32).view(torch.uint32)
    out = fbsr.fbsr_round_bits(x, "fp16", "src", k, words, scale=0.5)
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    w_pin, wh = gu.pinned_like(words)
    w_pin.copy_(words)
    o_pin, oh = gu.pinned_like(out)
    o_pin.copy_(out)
    torch.cuda.synchronize()
    piece_len = (1 << 20) // dpw * dpw                    # pieces start on word boundaries

    def piece(a, b):
        return gu.first_difference(oh[a:b], capi.fbsr_round_bits(xh[a:b], "fp16", "src", k, wh[a // dpw:(b + dpw - 1) // dpw], scale=0.5),
                                   a, "supplied bits")

    chk = gu.WholeTensorChecker(budget_s=60, piece=piece_len)
    _whole(n, "", piece, chk=chk)
    chk.report("supplied bits fp16 src k=3, 2^27")
    assert chk.fraction > 0.2


def test_run_time_format_and_binary8p4_full_size():
    n = 1 << 27
    x, scale = workloads.fp8_activations("b8p4", device="cuda")
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    desc = fbsr.format_desc(8, 4, 8, 0x7F, None, 0x80, True)              # float8_e4m3fnuz
    odesc = capi.make_desc(8, 4, 8, 0x7F, None, 0x80, True)
    got = fbsr.fbsr_round_desc(x, desc, "src", 3, seed=7, scale=scale)
    g_pin, gh = gu.pinned_like(got)
    g_pin.copy_(got)
    b8 = fbsr.fbsr_round(x, "b8p4", "src", 3, seed=7, scale=scale)
    b_pin, bh = gu.pinned_like(b8)
    b_pin.copy_(b8)
    torch.cuda.synchronize()

    def piece(a, b):
        return gu.first_difference(gh[a:b], capi.fbsr_round_desc(xh[a:b], odesc, "src", 3, seed=7, offset=a, scale=scale), a, "run-time format") or \
            gu.first_difference(bh[a:b], capi.fbsr_round(xh[a:b], "b8p4", "src", 3, seed=7, offset=a, scale=scale), a, "Binary8P4")

    _whole(n, "run-time (8,4,8;240) and Binary8P4, 2 x 2^27", piece)


def test_algorithm_1_steps_full_size():
    """fbsr_qat_update and fbsr_qat_adamw_step on 2^27 Binary8P4 weights with BFloat16 updates / gradients, 3 random
    bits: weights (and moments) of every parameter."""
    n = 1 << 27
    g = torch.Generator(device="cuda").manual_seed(21)
    w0 = fbsr.fbsr_round(torch.randn(n, device="cuda", generator=g), "b8p4", "rtne", 1, seed=0)
    u16 = (torch.randn(n, device="cuda", generator=g) * 1e-2).to(torch.bfloat16).view(torch.uint16)
    m0 = torch.randn(n, device="cuda", generator=g) * 1e-3
    v0 = torch.rand(n, device="cuda", generator=g) * 1e-4
    hyper = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    w1 = fbsr.fbsr_qat_update(w0.clone(), u16, "b8p4", "bf16", "src", 3, seed=8)
    w2, m2, v2 = w0.clone(), m0.clone(), v0.clone()
    fbsr.fbsr_qat_adamw_step(w2, u16, m2, v2, "b8p4", "bf16", "src", 3, seed=9, offset=0, step=3, **hyper)
    host = {}
    for name, t in (("w0", w0), ("u16", u16), ("m0", m0), ("v0", v0), ("w1", w1), ("w2", w2), ("m2", m2), ("v2", v2)):
        pin, arr = gu.pinned_like(t)
        pin.copy_(t)
        host[name] = (pin, arr)
    torch.cuda.synchronize()
    h = {k: v[1] for k, v in host.items()}

    def piece(a, b):
        e1 = capi.qat_update(h["w0"][a:b].copy(), h["u16"][a:b], "b8p4", "bf16", "src", 3, seed=8, offset=a)
        wb, mb, vb = h["w0"][a:b].copy(), h["m0"][a:b].copy(), h["v0"][a:b].copy()
        capi.qat_adamw_step(wb, h["u16"][a:b], mb, vb, "b8p4", "bf16", "src", 3, seed=9, offset=a, step=3, **hyper)
        return gu.first_difference(h["w1"][a:b], e1, a, "16-bit-sum update") or \
            gu.first_difference(h["w2"][a:b], wb, a, "fused step weights") or \
            gu.first_difference(h["m2"][a:b].view(np.uint32), mb.view(np.uint32), a, "fused step m") or \
            gu.first_difference(h["v2"][a:b].view(np.uint32), vb.view(np.uint32), a, "fused step v")

    _whole(n, "Algorithm-1 steps, 2^27 parameters", piece)
