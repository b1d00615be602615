"""Seeded synthetic inputs shaped like the paper's workloads.

Input generation only: nothing in this module performs or depends on the
rounding method.  Both the CUDA path and the CPU oracle consume the tensors
produced here (the oracle through a host copy of the same buffer).
"""
import math

import torch

FORMAT_MAX = {"bf16": 3.3895313892515355e38, "fp16": 65504.0, "e4m3": 448.0, "e5m2": 57344.0, "b8p4": 224.0}
FORMAT_MIN_NORMAL = {"bf16": 2.0 ** -126, "fp16": 2.0 ** -14, "e4m3": 2.0 ** -6, "e5m2": 2.0 ** -14, "b8p4": 2.0 ** -7}


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def bias_grid(cell_centred=True, points=1024, repeats=5000, device="cpu"):
    """Fig. 1 shape: `points` X values across the binade [1, 2), each repeated `repeats` times
    contiguously.  cell_centred=True puts X at the centres 1 + (2i+1)/(2 points) (values with four
    excess bits over bfloat16 whose mean error equals the continuous-input bias); False uses
    the grid 1 + i/points."""
    i = torch.arange(points, dtype=torch.float64)
    x = 1.0 + ((2 * i + 1) / (2 * points) if cell_centred else i / points)
    return x.to(torch.float32).repeat_interleave(repeats).to(device)


def fig2_grid(repeats=100_000, device="cpu"):
    """Fig. 2 shape: every BFloat16 value of the binade [1, 2) (128 codes), each repeated `repeats`
    times contiguously, as uint16 codes."""
    codes = torch.arange(0x3F80, 0x4000, dtype=torch.int32).to(torch.uint16)
    return codes.repeat_interleave(repeats).to(device)


def lp_sweep(n, src_fmt="bf16", seed=1234, device="cpu"):
    """The bandwidth-sweep distribution narrowed to a 16-bit source format (torch's nearest-even
    cast), as uint16 codes; magnitudes span 2^-12..2^12 so that both 8-bit targets see their normal,
    subnormal and saturating ranges."""
    g = _gen(seed, device)
    z = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    e = torch.rand(n, generator=g, device=device, dtype=torch.float32) * 24.0 - 12.0
    x = z * torch.exp2(e)
    dt = torch.bfloat16 if src_fmt == "bf16" else torch.float16
    return x.to(dt).view(torch.uint16)


def bandwidth_sweep(n, seed=1234, device="cpu"):
    """z ~ N(0, 1) times a log-uniform factor 2^U(-20, 20), per element."""
    g = _gen(seed, device)
    z = torch.randn(n, generator=g, device=device, dtype=torch.float32)
    e = torch.rand(n, generator=g, device=device, dtype=torch.float32) * 40.0 - 20.0
    return z * torch.exp2(e)


def fp8_activations(fmt, rows=4096, cols=32768, seed=7, device="cpu"):
    """Laplace(0, 1) activations with per-tensor amax scaling to the format's M, then 0.1 % of
    positions overwritten with values beyond the range, 0.1 % with values in and below the
    subnormal range, and 64 each of NaN, +Inf, -Inf.  Returns (x, scale)."""
    n = rows * cols
    g = _gen(seed, device)
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32) - 0.5
    x = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.49999997))
    amax = float(x.abs().max())
    scale = FORMAT_MAX[fmt] / amax
    k = max(n // 1000, 1)
    pos = torch.randperm(n, generator=g, device=device)
    over = pos[:k]
    sub = pos[k:2 * k]
    sgn = torch.where(torch.rand(k, generator=g, device=device) < 0.5, -1.0, 1.0)
    x[over] = sgn * (FORMAT_MAX[fmt] / scale) * (1.0 + 15.0 * torch.rand(k, generator=g, device=device))
    sgn = torch.where(torch.rand(k, generator=g, device=device) < 0.5, -1.0, 1.0)
    # magnitudes log-uniform over [2^-(P+5), 1) x min-normal: reaches below half the smallest subnormal
    span = {"e4m3": 9.0, "e5m2": 8.0, "fp16": 16.0, "bf16": 13.0, "b8p4": 9.0}[fmt]
    x[sub] = sgn * (FORMAT_MIN_NORMAL[fmt] / scale) * torch.exp2(-span * torch.rand(k, generator=g, device=device))
    s = min(64, max(n // 64, 1))
    sp = pos[2 * k:2 * k + 3 * s]
    x[sp[:s]] = float("nan")
    x[sp[s:2 * s]] = float("inf")
    x[sp[2 * s:3 * s]] = float("-inf")
    return x, float(torch.tensor(scale, dtype=torch.float32))


TRANSFORMER_BLOCK_SHAPES = [(4096, 4096), (4096, 11008)]


def optimizer_param_count(blocks=32):
    return blocks * sum(r * c for r, c in TRANSFORMER_BLOCK_SHAPES)


def optimizer_state(n, seed=99, device="cpu"):
    """Master weights ~ N(0, 0.02); zero moments."""
    g = _gen(seed, device)
    w = torch.randn(n, generator=g, device=device, dtype=torch.float32) * 0.02
    return w, torch.zeros_like(w), torch.zeros_like(w)


def optimizer_grad(n, step, device="cpu", out=None):
    """Gradient of step `step` (1-based) ~ N(0, 1e-3), torch seed 100 + step."""
    g = _gen(100 + step, device)
    if out is None:
        out = torch.empty(n, device=device, dtype=torch.float32)
    out.normal_(0.0, 1e-3, generator=g)
    return out


def accumulation_weights(n, seed=5, device="cpu"):
    """bfloat16 weights ~ N(0, 0.02) as uint16 codes (torch's nearest-even cast)."""
    g = _gen(seed, device)
    w = torch.randn(n, generator=g, device=device, dtype=torch.float32) * 0.02
    return w.to(torch.bfloat16).view(torch.uint16)


def accumulation_update(w_codes, step, magnitude=2.0 ** -12, seed=1000, device=None):
    """u = +-c * magnitude * ulp_bf16(w), c ~ U(0, 1], fair sign, fresh per step."""
    device = w_codes.device if device is None else device
    g = _gen(seed + step, device)
    w = w_codes.view(torch.bfloat16).to(torch.float32)
    _, ex = torch.frexp(w.abs())
    ulp = torch.ldexp(torch.ones_like(w), torch.clamp(ex - 1, min=-126) - 7)
    c = 1.0 - torch.rand(w.numel(), generator=g, device=device, dtype=torch.float32)
    sgn = torch.where(torch.rand(w.numel(), generator=g, device=device) < 0.5, -1.0, 1.0)
    return (sgn * c * magnitude * ulp).to(torch.float32)
