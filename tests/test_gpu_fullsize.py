"""Parity at the benchmark's full sizes, in the launch configuration bench.py times, over EVERY element:
each output is a pure function of the input element and its global index (Section II-A Eq. (5), Section II-B),
so the scalar oracle checks the whole tensor piece by piece on all host cores.  A time budget guards the
run against a slow host; if it ever cuts a leg short, the fraction that ran is printed and raised as a
warning (see gpu_util.WholeTensorChecker)."""
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
    capi.lib()
    module.fbsr, module.capi, module.gu, module.workloads = fbsr, capi, gpu_util, workloads


def test_bandwidth_sweep_full_size():
    """2^28 elements, every (format, variant, k) of the sweep: all 48 x 2^28 codes against the oracle."""
    n = 1 << 28
    x = workloads.bandwidth_sweep(n, seed=1234, device="cuda")
    out = torch.empty(n, dtype=torch.uint16, device="cuda")
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    out_pin, oh = gu.pinned_like(out)
    combos = [(f, v, k) for f in ("bf16", "fp16") for v in VARIANTS for k in (1, 2, 3, 4, 6, 8, 13, 16)]
    chk = gu.WholeTensorChecker(budget_s=420)
    for idx, (fmt, variant, k) in enumerate(combos):
        out.zero_()
        fbsr.fbsr_round(x, fmt, variant, k, seed=1234, offset=0, out=out)
        out_pin.copy_(out)
        torch.cuda.synchronize()

        def piece(a, b, fmt=fmt, variant=variant, k=k):
            expect = capi.fbsr_round(xh[a:b], fmt, variant, k, seed=1234, offset=a)
            return gu.first_difference(oh[a:b], expect, a, "%s %s k=%d" % (fmt, variant, k))

        chk.run(n, piece, remaining_calls=len(combos) - idx)
        if fmt == "bf16" and k == 16 and variant == "srff":
            # with all 16 bits the round-up frequency equals the mean fractional part
            bits = x.view(torch.int32)
            up = (out.view(torch.int16).to(torch.int32) & 0xFFFF) - ((bits >> 16) & 0xFFFF)
            frac = ((bits & 0xFFFF).double() / 65536.0).mean().item()
            assert abs(up.double().mean().item() - frac) < 2e-4
            del bits, up
    chk.report("bandwidth sweep, 48 x 2^28")
    assert chk.fraction > 0.2


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_activations_full_size(fmt):
    """4096 x 32768 Laplace activations with outliers, subnormals, NaN and Inf; k in {2, 4, 8}, every variant:
    all 9 x 2^27 codes against the oracle."""
    x, scale = workloads.fp8_activations(fmt, device="cuda")
    n = x.numel()
    out = torch.empty(n, dtype=torch.uint8, device="cuda")
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    out_pin, oh = gu.pinned_like(out)
    combos = [(k, v) for k in (2, 4, 8) for v in VARIANTS]
    chk = gu.WholeTensorChecker(budget_s=90)
    for idx, (k, variant) in enumerate(combos):
        out.zero_()
        fbsr.fbsr_round(x, fmt, variant, k, seed=7, scale=scale, out=out)
        out_pin.copy_(out)
        torch.cuda.synchronize()

        def piece(a, b, k=k, variant=variant):
            expect = capi.fbsr_round(xh[a:b], fmt, variant, k, seed=7, offset=a, scale=scale)
            return gu.first_difference(oh[a:b], expect, a, "%s %s k=%d" % (fmt, variant, k))

        chk.run(n, piece, remaining_calls=len(combos) - idx)
    chk.report("fp8 activations %s, 9 x 2^27" % fmt)
    assert chk.fraction > 0.2
    # whole-tensor counts of the special paths
    codes = fbsr.fbsr_round(x, fmt, "srf", 4, seed=7, scale=scale)
    mag = codes & 0x7F
    nan_code, max_code = 0x7F, (0x7E if fmt == "e4m3" else 0x7B)
    assert int((mag == nan_code).sum()) == 64
    assert int((mag == max_code).sum()) >= 2000
    if fmt == "e5m2":
        assert int((mag == 0x7C).sum()) == 128


def _k_of_step(step):
    return (2, 4, 8)[(step // 4) % 3]          # step 1 -> 2, steps 4..7 -> 4, steps 8..10 -> 8


@pytest.mark.parametrize("algo", ["sgd", "adam"])
def test_fused_optimizer_full_size(algo):
    """The 32-block parameter list (1 979 711 488 fp32 parameters), 10 steps with step-indexed seeds, k in {2, 4, 8}.
    Steps 1 and 10 are checked in full -- master weights, moments and bf16 codes of every parameter -- against the
    oracle applied to the state the GPU held before that step; a set of slices is followed through all 10 steps."""
    n = workloads.optimizer_param_count(32)
    rng = np.random.default_rng(5)
    slices = [(0, 4096), (n - 4096, n)] + [(int(s), int(s) + 4096) for s in rng.integers(0, n - 4096, size=4)]
    variant = "srf" if algo == "sgd" else "src"
    w, m, v = workloads.optimizer_state(n, device="cuda")
    if algo == "sgd":
        v = None
    state = [t for t in (w, m, v) if t is not None]
    g = torch.empty(n, dtype=torch.float32, device="cuda")
    lp = torch.empty(n, dtype=torch.uint16, device="cuda")
    prev = [torch.empty_like(t) for t in state]
    host = [[t[a:b].cpu().numpy().copy() for t in state] for a, b in slices]
    slab = 1 << 26
    pins = {name: gu.pinned_like(torch.empty(slab, dtype=torch.float32)) for name in
            ["g"] + ["prev%d" % i for i in range(len(state))] + ["new%d" % i for i in range(len(state))]}
    pins["lp"] = gu.pinned_like(torch.empty(slab, dtype=torch.uint16))
    chk = gu.WholeTensorChecker(budget_s=200)
    n_slabs = -(-n // slab)

    def oracle_step(step, k, arrays, gh, offset):
        if algo == "sgd":
            return capi.sgd_update(arrays[0], gh, arrays[1], "bf16", variant, k, seed=50 + step, offset=offset,
                                   lr=1e-4, mu=0.9)
        return capi.adam_update(arrays[0], gh, arrays[1], arrays[2], "bf16", variant, k, seed=50 + step, offset=offset,
                                lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, step=step)

    for step in range(1, 11):
        workloads.optimizer_grad(n, step, device="cuda", out=g)
        k = _k_of_step(step)
        full = step in (1, 10)
        if full:
            for p, t in zip(prev, state):
                p.copy_(t)
        if algo == "sgd":
            fbsr.fbsr_sgd_update(w, g, m, "bf16", variant, k, seed=50 + step, offset=0, lr=1e-4, mu=0.9, out=lp)
        else:
            fbsr.fbsr_adam_update(w, g, m, v, "bf16", variant, k, seed=50 + step, offset=0, lr=1e-4, beta1=0.9,
                                  beta2=0.999, eps=1e-8, step=step, out=lp)
        # the slices' own trajectory, every step
        for (a, b), arrays in zip(slices, host):
            e = oracle_step(step, k, arrays, g[a:b].cpu().numpy(), a)
            gu.assert_codes_equal(lp[a:b], e, "%s step %d slice %d" % (algo, step, a))
            for t, h in zip(state, arrays):
                assert np.array_equal(t[a:b].cpu().numpy().view(np.uint32), h.view(np.uint32))
        if not full:
            continue
        # every parameter, one slab at a time through pinned staging
        for s in range(n_slabs):
            a0, b0 = s * slab, min(n, (s + 1) * slab)
            ln = b0 - a0
            pins["g"][0][:ln].copy_(g[a0:b0], non_blocking=True)
            pins["lp"][0][:ln].copy_(lp[a0:b0], non_blocking=True)
            for i, (p, t) in enumerate(zip(prev, state)):
                pins["prev%d" % i][0][:ln].copy_(p[a0:b0], non_blocking=True)
                pins["new%d" % i][0][:ln].copy_(t[a0:b0], non_blocking=True)
            torch.cuda.synchronize()

            def piece(a, b, a0=a0, step=step, k=k):
                arrays = [pins["prev%d" % i][1][a:b] for i in range(len(state))]      # updated in place by the oracle
                e = oracle_step(step, k, arrays, pins["g"][1][a:b], a0 + a)
                msg = gu.first_difference(pins["lp"][1][a:b], e, a0 + a, "%s step %d codes" % (algo, step))
                for i, name in enumerate(("w", "m", "v")[: len(state)]):
                    msg = msg or gu.first_difference(pins["new%d" % i][1][a:b].view(np.uint32), arrays[i].view(np.uint32),
                                                     a0 + a, "%s step %d %s" % (algo, step, name))
                return msg

            remaining = (n_slabs - s) + (n_slabs if step == 1 else 0)
            chk.run(ln, piece, remaining_calls=remaining)
    chk.report("fused %s, steps 1 and 10 of 10, 1 979 711 488 parameters" % algo)
    assert chk.fraction > 0.2


@pytest.mark.parametrize("variant", VARIANTS)
def test_small_update_accumulation_full_size(variant):
    """2^24 bfloat16 weights, 1000 updates of at most 2^-12 ulp, k in {1, 2, 4}: steps 1-10 and every 100th are
    checked in full against the oracle applied to the GPU's previous state; drift of mean |w| against the exact
    fp64 accumulation (Section IV: stagnation for the unbiased predicates, a systematic shrink for SRFF)."""
    n = 1 << 24
    steps = 1000
    w0 = workloads.accumulation_weights(n, device="cuda")
    checked = set(range(1, 11)) | set(range(100, steps + 1, 100))
    before_pin, before_h = gu.pinned_like(w0)
    after_pin, after_h = gu.pinned_like(w0)
    u_pin, u_h = gu.pinned_like(torch.empty(n, dtype=torch.float32))
    chk = gu.WholeTensorChecker(budget_s=90)
    todo = 3 * len(checked)
    for k in (1, 2, 4):
        w = w0.clone()
        exact = w0.view(torch.bfloat16).double()
        for step in range(1, steps + 1):
            u = workloads.accumulation_update(w, step)
            exact += u.double()
            if step in checked:
                before_pin.copy_(w)
                u_pin.copy_(u)
            fbsr.fbsr_accumulate(w, u, "bf16", variant, k, seed=step, offset=0)
            if step in checked:
                after_pin.copy_(w)
                torch.cuda.synchronize()

                def piece(a, b, k=k, step=step):
                    expect = capi.accumulate(before_h[a:b].copy(), u_h[a:b], "bf16", variant, k, seed=step, offset=a)
                    return gu.first_difference(after_h[a:b], expect, a, "%s k=%d step %d" % (variant, k, step))

                chk.run(n, piece, remaining_calls=todo)
                todo -= 1
        drift = (w.view(torch.bfloat16).double().abs().mean() - exact.abs().mean()).item()
        scale = w0.view(torch.bfloat16).double().abs().mean().item()
        moved = float((w != w0).double().mean())
        print("accumulation %s k=%d: relative drift of mean|w| %.3e, weights moved %.4f" % (variant, k, drift / scale, moved))
        if variant == "srff":
            assert drift < -1e-2 * scale * 2.0 ** -k        # systematic shrink of |w| (bias toward zero)
            assert moved > 0.5
        else:
            assert abs(drift) < 1e-6 * scale                # weights do not move; only the tiny exact sum differs
            assert moved == 0.0
    chk.report("accumulation %s, 20 of 1000 steps x 3 draw widths x 2^24" % variant)
    assert chk.fraction > 0.2


@pytest.mark.parametrize("fmt,variant,k,data", [("bf16", "srf", 2, "sweep"), ("fp16", "src", 3, "sweep"), ("e4m3", "srf", 3, "fp8act")])
def test_statistics_full_size(fmt, variant, k, data):
    """The fused error statistics at the benchmark's sizes: counts equal and binary64 sums within 1e-9 of the oracle's
    over every element (the oracle's per-piece totals added with an exact sum), codes included."""
    import math
    import threading
    if data == "sweep":
        x, scale = workloads.bandwidth_sweep(1 << 28, seed=1234, device="cuda"), 1.0
    else:
        x, scale = workloads.fp8_activations(fmt, device="cuda")
    n = x.numel()
    codes, st, _, _ = fbsr.fbsr_round_stats(x, fmt, variant, k, seed=1234, offset=0, scale=scale)
    again = fbsr.fbsr_round_stats(x, fmt, variant, k, seed=1234, offset=0, scale=scale)[1]
    assert again == st                                   # reproducible bit for bit
    x_pin, xh = gu.pinned_like(x)
    x_pin.copy_(x)
    c_pin, ch = gu.pinned_like(codes)
    c_pin.copy_(codes)
    torch.cuda.synchronize()
    pieces, lock = [], threading.Lock()

    def piece(a, b):
        ecodes, est, _, _ = capi.fbsr_round_stats(xh[a:b], fmt, variant, k, seed=1234, offset=a, scale=scale)
        with lock:
            pieces.append(est)
        return gu.first_difference(ch[a:b], ecodes, a, "%s %s k=%d statistics codes" % (fmt, variant, k))

    chk = gu.WholeTensorChecker(budget_s=120)
    chk.run(n, piece)
    chk.report("statistics %s %s k=%d, 2^%d elements" % (fmt, variant, k, n.bit_length() - 1))
    assert chk.fraction == 1.0                           # totals need every piece
    for key in ("n_finite", "n_up", "n_nan", "n_inf", "n_sat"):
        assert st[key] == sum(p[key] for p in pieces), key
    sum_abs = math.fsum(p["sum_abs_e"] for p in pieces)
    for key in ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e"):
        want = math.fsum(p[key] for p in pieces)
        assert abs(st[key] - want) <= 1e-9 * max(abs(want), 1e-3 * sum_abs), (key, st[key], want)
