"""One small, self-contained invocation of a single kernel, for profilers and quick timing.

    python -m paper_2504_20634_b200.profile_case --op round --fmt bf16 --variant srf --k 4 --log2n 26 --iters 5

Inputs are the synthetic 'bandwidth sweep' distribution (seed 1234).  Prints the mean
CUDA-event time per launch and the algorithmic bandwidth.  With --log2n 26 the case holds
well under 1 GiB on the device and still exceeds the L2 capacity.
"""
import argparse
import json

import torch

import paper_2504_20634_b200 as fbsr
from paper_2504_20634_b200 import workloads


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="round", choices=["round", "sgd", "adam", "accumulate", "stats", "bits", "lp", "mx", "desc", "qat", "qat_adamw"])
    ap.add_argument("--src-fmt", default="bf16", help="source format for --op lp")
    ap.add_argument("--fmt", default="bf16")
    ap.add_argument("--variant", default="srf")
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--log2n", type=int, default=26)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=2)
    ap.add_argument("--data", default="sweep", choices=["sweep", "fp8act"],
                    help="sweep: N(0,1) x 2^U(-20,20); fp8act: Laplace activations with amax scaling and injected outliers (8-bit formats)")
    ap.add_argument("--scale", type=float, default=1.0, help="per-tensor scale for --op round / stats on the sweep data")
    ap.add_argument("--misalign", type=int, default=0, help="start the source this many elements off its allocation (--op round)")
    args = ap.parse_args()

    n = 1 << args.log2n
    dev = torch.device("cuda", 0)
    scale = args.scale
    base_fmt = args.fmt.split("+")[0]               # "fp16+ieee": the IEEE overflow option
    if args.data == "fp8act":
        x, scale = workloads.fp8_activations(base_fmt, rows=n // 32768, cols=32768, device=dev)
    elif args.misalign:
        x = workloads.bandwidth_sweep(n + args.misalign, seed=1234, device=dev)[args.misalign:]
    else:
        x = workloads.bandwidth_sweep(n, seed=1234, device=dev)
    code_bytes = 2 if base_fmt in ("bf16", "fp16") else 1
    out = torch.empty(n, dtype=fbsr.CODE_DTYPE[base_fmt], device=dev)
    if args.op == "round":
        bytes_per_elem = 4 + code_bytes
        run = lambda s: fbsr.fbsr_round(x, args.fmt, args.variant, args.k, seed=1234, scale=scale, out=out)
    elif args.op == "desc":
        # the same format, handed over as a run-time descriptor (general kernel)
        desc = fbsr.format_desc(*{"bf16": (16, 8, 127, 0x7F7F, 0x7F80, 0x7FC0, False),
                                  "fp16": (16, 11, 15, 0x7BFF, 0x7C00, 0x7E00, False),
                                  "e4m3": (8, 4, 7, 0x7E, None, 0x7F, False),
                                  "e5m2": (8, 3, 15, 0x7B, 0x7C, 0x7F, False),
                                  "b8p4": (8, 4, 8, 0x7E, 0x7F, 0x80, True)}[args.fmt])
        bytes_per_elem = 4 + code_bytes
        run = lambda s: fbsr.fbsr_round_desc(x, desc, args.variant, args.k, seed=1234, out=out)
    elif args.op == "qat_adamw":
        # Algorithm 1 fused: 8-bit weights in place, 16-bit gradients, binary32 moments: 20 B/parameter
        fbsr.fbsr_round(x.mul(2.0 ** -18).clamp_(-3, 3), args.fmt, "rtne", 1, seed=0, out=out)
        g16 = (torch.randn(n, device=dev) * 1e-2).to(torch.bfloat16 if args.src_fmt == "bf16" else torch.float16).view(torch.uint16)
        m, v = torch.zeros(n, device=dev), torch.zeros(n, device=dev)
        bytes_per_elem = 20
        run = lambda s: fbsr.fbsr_qat_adamw_step(out, g16, m, v, args.fmt, args.src_fmt, args.variant, args.k, s, 0,
                                                 1e-3, 0.9, 0.95, 1e-8, 0.1, s + 1)
    elif args.op == "qat":
        # last line of Algorithm 1 with the 16-bit sum: 8-bit weights in place, 16-bit updates: 4 B/element
        fbsr.fbsr_round(x.mul(2.0 ** -18).clamp_(-3, 3), base_fmt, "rtne", 1, seed=0, out=out)
        u16 = (torch.randn(n, device=dev) * 1e-2).to(torch.bfloat16 if args.src_fmt == "bf16" else torch.float16).view(torch.uint16)
        bytes_per_elem = 4
        run = lambda s: fbsr.fbsr_qat_update(out, u16, args.fmt, args.src_fmt, args.variant, args.k, seed=s)
    elif args.op == "lp":
        codes = workloads.lp_sweep(n, args.src_fmt, device=dev)
        bytes_per_elem = 2 + code_bytes
        run = lambda s: fbsr.fbsr_round_lp(codes, args.src_fmt, args.fmt, args.variant, args.k, seed=1234, out=out)
    elif args.op == "mx":
        scales = torch.empty((n + 31) // 32, dtype=torch.uint8, device=dev)
        bytes_per_elem = 4 + code_bytes + 1.0 / 32
        run = lambda s: fbsr.fbsr_round_mx(x, args.fmt, args.variant, args.k, seed=1234, out=out, scales=scales)
    elif args.op == "bits":
        dpw = 32 // args.k
        words = torch.randint(0, 2 ** 31, ((n + dpw - 1) // dpw,), device=dev, dtype=torch.int32).view(torch.uint32)
        bytes_per_elem = 4 + code_bytes + 4.0 / dpw
        run = lambda s: fbsr.fbsr_round_bits(x, args.fmt, args.variant, args.k, words, out=out)
    elif args.op == "stats":
        bytes_per_elem = 4 + code_bytes
        ws = torch.empty(fbsr.fbsr_stats_workspace_bytes(), dtype=torch.uint8, device=dev)
        total = torch.empty(72, dtype=torch.uint8, device=dev)
        run = lambda s: fbsr.fbsr_round_stats(x, args.fmt, args.variant, args.k, seed=1234, scale=scale, out=out,
                                              workspace=ws, total=total, read_back=False)
    elif args.op == "accumulate":
        x.mul_(1e-3)
        out.copy_(workloads.accumulation_weights(n, device=dev) if args.fmt == "bf16" else torch.zeros_like(out))
        bytes_per_elem = 4 + 2 * code_bytes
        run = lambda s: fbsr.fbsr_accumulate(out, x, args.fmt, args.variant, args.k, seed=s)
    else:
        w, m, v = workloads.optimizer_state(n, device=dev)
        g = workloads.optimizer_grad(n, 1, device=dev)
        if args.op == "sgd":
            bytes_per_elem = 20 + code_bytes
            run = lambda s: fbsr.fbsr_sgd_update(w, g, m, args.fmt, args.variant, args.k, s, 0, 1e-4, 0.9, out=out)
        else:
            bytes_per_elem = 28 + code_bytes
            run = lambda s: fbsr.fbsr_adam_update(w, g, m, v, args.fmt, args.variant, args.k, s, 0, 1e-4, 0.9, 0.999,
                                                  1e-8, s, out=out)
    for s in range(1, args.warmup + 1):
        run(s)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for s in range(args.iters):
        run(args.warmup + 1 + s)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.iters
    print(json.dumps({"op": args.op, "fmt": args.fmt, "variant": args.variant, "k": args.k, "n": n, "data": args.data, "scale": scale,
                      "ms_per_launch": ms, "GB/s": bytes_per_elem * n / (ms * 1e-3) / 1e9,
                      "Gelem/s": n / (ms * 1e-3) / 1e9}))


if __name__ == "__main__":
    main()
