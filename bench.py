#!/usr/bin/env python
"""Benchmark of the few-bit stochastic rounding path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload ("bandwidth sweep"): 2^28 binary32 elements per GPU, z ~ N(0,1) x 2^U(-20,20), seed 1234,
resident in HBM.  One step rounds the tensor to bfloat16 and to binary16 for every
k in {1,2,3,4,6,8,13,16} and every variant (SRFF, SRF, SRC): 48 fbsr_round launches.
Metric: elements rounded per second over the whole job (Gelem/s).

Prints one JSON line (rank 0).  `--impl reference` times the scalar CPU oracle on a bounded
sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_ELEMS = 1 << 28
K_LIST = (1, 2, 3, 4, 6, 8, 13, 16)
FMT_LIST = ("bf16", "fp16")
VARIANT_LIST = ("srff", "srf", "src")
SEED = 1234
BYTES_PER_ELEM = 6.0            # 4 read + 2 written, both 16-bit targets
METRIC = "fbsr_round throughput, fp32->bf16/fp16, all k and variants"
UNIT = "Gelem/s"


def sweep():
    return [(f, v, k) for f in FMT_LIST for v in VARIANT_LIST for k in K_LIST]


# DRAM traffic of one 2^28-element bf16 launch, from the ncu capture summarised in
# profiles/tile_kernel_round.txt (dram__bytes_read.sum + dram__bytes_write.sum of a 2^27-element
# launch, scaled by the elements processed).  Valid only for the kernel sources it was taken from.
TRAFFIC_BYTES_PER_LAUNCH = 2 * (536.893952e6 + 221.408768e6)
TRAFFIC_KERNEL_SHA = "358d6c0691e7a25d"


def kernel_source_sha():
    import hashlib
    h = hashlib.sha256()
    for name in ("fbsr_device.cuh", "fbsr_kernels.cuh"):
        with open(os.path.join(ROOT, "paper_2504_20634_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm = sorted(float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit())
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) >= 9:
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def time_oracle(x_host, combos, offset, threads):
    """Oracle wall time over `combos` on the host slice, split over `threads` disjoint chunks."""
    import concurrent.futures
    from oracle import capi
    capi.lib()
    n = x_host.size
    cuts = [n * i // threads for i in range(threads + 1)]

    def work(i):
        a, b = cuts[i], cuts[i + 1]
        for fmt, variant, k in combos:
            capi.fbsr_round(x_host[a:b], fmt, variant, k, seed=SEED, offset=offset + a)

    t0 = time.perf_counter()
    if threads == 1:
        work(0)
    else:
        with concurrent.futures.ThreadPoolExecutor(threads) as pool:
            list(pool.map(work, range(threads)))
    return time.perf_counter() - t0


def run_reference(args, rank, world):
    """The scalar oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    from paper_2504_20634_b200 import workloads
    sample = 1 << 19
    x = workloads.bandwidth_sweep(sample, seed=SEED, device="cpu").numpy()
    combos = sweep()
    for _ in range(args.warmup):
        time_oracle(x[: sample // 8], combos[:6], 0, 1)
    t = 0.0
    for _ in range(args.steps):
        t += time_oracle(x, combos, 0, 1)
    value = sample * len(combos) * args.steps / t / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": "bandwidth sweep (2^28 fp32 -> bf16, fp16; k in {1,2,3,4,6,8,13,16}; SRFF/SRF/SRC; seed 1234)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "first 2^19 elements of the sweep tensor, all 48 (format, variant, k) combinations per step"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--skip-extras", action="store_true", help="skip the per-kernel table and the fused-optimizer timing")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import paper_2504_20634_b200 as fbsr            # raises if libfbsr.so is missing: no fallback
    from paper_2504_20634_b200 import sharding, workloads

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- inputs: this rank's shard of a world * 2^28 element tensor (weak scaling); shard boundaries sit
    # on a multiple of every tile size, global index of local element i = offset + i
    offset, shard_end = sharding.my_shard(world * N_ELEMS, rank, world)
    n_local = shard_end - offset
    x = workloads.bandwidth_sweep(n_local, seed=SEED + rank, device=dev)
    out = torch.empty(n_local, dtype=torch.uint16, device=dev)
    combos = sweep()
    stream = torch.cuda.current_stream(dev)

    def step():
        for fmt, variant, k in combos:
            fbsr.fbsr_round(x, fmt, variant, k, seed=SEED, offset=offset, out=out)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = fbsr.fbsr_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    launches = fbsr.fbsr_launch_count() - launches0
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    ms = sharding.max_over_ranks(ms, dist, dev)
    launches = int(sharding.sum_over_ranks(int(launches), dist, dev))
    ms_per_step = ms / args.steps
    total_elems = float(N_ELEMS) * len(combos) * world
    value = total_elems / (ms_per_step * 1e-3) / 1e9

    # ---- roofline of the tiled rounding kernel: all 48 launches move 6 B/element
    peak, peak_kind = measured_peak_gbs()
    achieved = BYTES_PER_ELEM * n_local * len(combos) / (ms_per_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": TRAFFIC_BYTES_PER_LAUNCH if kernel_source_sha() == TRAFFIC_KERNEL_SHA else None,
                "peak_source": peak_kind + " copy bandwidth",
                "kernel": "fbsr::tile_kernel<RoundOp, fmt, variant, k> (average over the 48 launches of a step)",
                "algorithmic_bytes_per_launch": BYTES_PER_ELEM * n_local,
                "frac_of_8TBps": achieved / 8000.0}

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    e2e = None
    cpu_baseline = None
    extras = {}
    if rank == 0 or world > 1:
        n_e2e = 1 << 26
        e2e_combos = combos
        src_h = torch.empty(n_e2e, dtype=torch.float32).pin_memory()
        src_h.copy_(x[:n_e2e])
        dst_h = torch.empty(n_e2e, dtype=torch.uint16).pin_memory()
        ws = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

        def e2e_step():
            for fmt, variant, k in e2e_combos:
                fbsr.fbsr_round_host(src_h, dst_h, fmt, variant, k, SEED, offset, 1.0, ws)
            stream.synchronize()
            return int(dst_h[-1])          # the step's result is read on the host

        e2e_step()
        barrier()
        e2e_steps = max(1, min(args.steps, 3))
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        t1.record(stream)
        barrier()
        e_ms = t0.elapsed_time(t1)
        e_ms = sharding.max_over_ranks(e_ms, dist, dev)
        e_val = float(n_e2e) * len(e2e_combos) * e2e_steps * world / (e_ms * 1e-3) / 1e9
        e2e = {"value": e_val, "unit": UNIT, "h2d_bytes_per_step": 4 * n_e2e * len(e2e_combos),
               "d2h_bytes_per_step": 2 * n_e2e * len(e2e_combos),
               "note": "fbsr_round_host on a 2^26-element pinned host slice of the same tensor, 48 calls per step, %d steps" % e2e_steps}
        del src_h, dst_h, ws

    if rank == 0 and not args.skip_extras:
        # per-launch table (one pass, events around every launch; not part of the timed region)
        table = {}
        evs = []
        for fmt, variant, k in combos:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fbsr.fbsr_round(x, fmt, variant, k, seed=SEED, offset=offset, out=out)      # untimed first launch
            a.record(stream)
            for _ in range(3):
                fbsr.fbsr_round(x, fmt, variant, k, seed=SEED, offset=offset, out=out)
            b.record(stream)
            evs.append((fmt, variant, k, a, b))
        torch.cuda.synchronize()
        for fmt, variant, k, a, b in evs:
            table["%s/%s/k%d" % (fmt, variant, k)] = round(BYTES_PER_ELEM * n_local / (a.elapsed_time(b) / 3 * 1e-3) / 1e9, 1)
        extras["round_GBps"] = table
        # fp8 leg of the metric (5 B/element), 2^27 elements
        x8 = x[: 1 << 27]
        out8 = torch.empty(1 << 27, dtype=torch.uint8, device=dev)
        t8 = {}
        for fmt in ("e4m3", "e5m2", "b8p4"):
            for k in (2, 4, 8):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                for _ in range(3):
                    fbsr.fbsr_round(x8, fmt, "srf", k, seed=7, scale=2.0 ** -10, out=out8)
                a.record(stream)
                for _ in range(10):
                    fbsr.fbsr_round(x8, fmt, "srf", k, seed=7, scale=2.0 ** -10, out=out8)
                b.record(stream)
                torch.cuda.synchronize()
                t8["%s/srf/k%d" % (fmt, k)] = round(5.0 * (1 << 27) / (a.elapsed_time(b) / 10 * 1e-3) / 1e9, 1)
        extras["round_fp8_GBps"] = t8
        # rounding with the fused error statistics (the call reads the totals back, so each iteration synchronises)
        ts = {}
        for fmt, k in (("bf16", 2), ("e4m3", 3)):
            cb = 2 if fmt == "bf16" else 1
            outs = torch.empty(1 << 27, dtype=fbsr.CODE_DTYPE[fmt], device=dev)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fbsr.fbsr_round_stats(x8, fmt, "srf", k, seed=7, scale=2.0 ** -10, out=outs)
            a.record(stream)
            for _ in range(5):
                fbsr.fbsr_round_stats(x8, fmt, "srf", k, seed=7, scale=2.0 ** -10, out=outs)
            b.record(stream)
            torch.cuda.synchronize()
            ts["%s/srf/k%d" % (fmt, k)] = round((4.0 + cb) * (1 << 27) / (a.elapsed_time(b) / 5 * 1e-3) / 1e9, 1)
            del outs
        extras["round_stats_GBps"] = ts
        # a format described at run time (general kernel): float8_e4m3fnuz = (8, 4, 8; 240), 5 B/element
        desc = fbsr.format_desc(8, 4, 8, 0x7F, None, 0x80, True)
        td = {}
        for k in (3, 8):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            fbsr.fbsr_round_desc(x8, desc, "srf", k, seed=7, scale=2.0 ** -10, out=out8)
            a.record(stream)
            for _ in range(5):
                fbsr.fbsr_round_desc(x8, desc, "srf", k, seed=7, scale=2.0 ** -10, out=out8)
            b.record(stream)
            torch.cuda.synchronize()
            td["(8,4,8;240)/srf/k%d" % k] = round(5.0 * (1 << 27) / (a.elapsed_time(b) / 5 * 1e-3) / 1e9, 1)
        extras["round_desc_GBps"] = td
        del x8, out8
        # 16-bit sources into 8-bit formats (3 B/element) and the 16-bit-sum weight update (4 B/element)
        codes16 = workloads.lp_sweep(n_local, "bf16", device=dev)
        w8 = torch.empty(n_local, dtype=torch.uint8, device=dev)
        tlp = {}
        for fmt in ("e4m3", "e5m2", "b8p4"):
            for variant in VARIANT_LIST:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                fbsr.fbsr_round_lp(codes16, "bf16", fmt, variant, 3, seed=SEED, out=w8)
                a.record(stream)
                for _ in range(10):
                    fbsr.fbsr_round_lp(codes16, "bf16", fmt, variant, 3, seed=SEED, out=w8)
                b.record(stream)
                torch.cuda.synchronize()
                tlp["bf16->%s/%s/k3" % (fmt, variant)] = round(3.0 * n_local / (a.elapsed_time(b) / 10 * 1e-3) / 1e9, 1)
        extras["round_lp_GBps"] = tlp
        fbsr.fbsr_round_lp(codes16, "bf16", "e4m3", "rtne", 1, seed=0, out=w8)
        upd = (torch.randn(n_local, device=dev) * 0.01).to(torch.bfloat16).view(torch.uint16)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fbsr.fbsr_qat_update(w8, upd, "e4m3", "bf16", "src", 3, seed=1)
        a.record(stream)
        for s_ in range(10):
            fbsr.fbsr_qat_update(w8, upd, "e4m3", "bf16", "src", 3, seed=2 + s_)
        b.record(stream)
        torch.cuda.synchronize()
        extras["qat_update_e4m3_bf16_src_k3_GBps"] = round(4.0 * n_local / (a.elapsed_time(b) / 10 * 1e-3) / 1e9, 1)
        # the same step in Section IV's own format (Binary8P4 weights)
        fbsr.fbsr_round_lp(codes16, "bf16", "b8p4", "rtne", 1, seed=0, out=w8)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fbsr.fbsr_qat_update(w8, upd, "b8p4", "bf16", "src", 3, seed=1)
        a.record(stream)
        for s_ in range(10):
            fbsr.fbsr_qat_update(w8, upd, "b8p4", "bf16", "src", 3, seed=2 + s_)
        b.record(stream)
        torch.cuda.synchronize()
        extras["qat_update_b8p4_bf16_src_k3_GBps"] = round(4.0 * n_local / (a.elapsed_time(b) / 10 * 1e-3) / 1e9, 1)
        # one whole iteration of Algorithm 1, fused (20 B/parameter): Binary8P4 weights, bf16 gradients, 3 random bits
        grad16 = upd
        m_ = torch.zeros(n_local, device=dev)
        v_ = torch.zeros(n_local, device=dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fbsr.fbsr_qat_adamw_step(w8, grad16, m_, v_, "b8p4", "bf16", "src", 3, 1, 0, 1e-3, 0.9, 0.95, 1e-8, 0.1, 1)
        a.record(stream)
        for s_ in range(10):
            fbsr.fbsr_qat_adamw_step(w8, grad16, m_, v_, "b8p4", "bf16", "src", 3, 2 + s_, 0, 1e-3, 0.9, 0.95, 1e-8, 0.1, 2 + s_)
        b.record(stream)
        torch.cuda.synchronize()
        ms_ = a.elapsed_time(b) / 10
        extras["qat_adamw_step_b8p4_bf16_src_k3"] = {"Gparam/s": round(n_local / (ms_ * 1e-3) / 1e9, 2),
                                                      "GB/s": round(20.0 * n_local / (ms_ * 1e-3) / 1e9, 1)}
        del codes16, w8, upd, grad16, m_, v_
        # fused optimizer step on the 32-block parameter list (22 B/param SGD-momentum, 30 B/param Adam)
        try:
            n_p = workloads.optimizer_param_count(32)
            w, m, v = workloads.optimizer_state(n_p, device=dev)
            g = workloads.optimizer_grad(n_p, 1, device=dev)
            lp = torch.empty(n_p, dtype=torch.uint16, device=dev)
            opt = {}
            for name, fn, bpp in (("sgd_momentum", lambda s: fbsr.fbsr_sgd_update(w, g, m, "bf16", "srf", 4, SEED + s, 0, 1e-4, 0.9, out=lp), 22.0),
                                  ("adam", lambda s: fbsr.fbsr_adam_update(w, g, m, v, "bf16", "srf", 4, SEED + s, 0, 1e-4, 0.9, 0.999, 1e-8, s, out=lp), 30.0)):
                fn(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for s in range(2, 7):
                    fn(s)
                b.record(stream)
                torch.cuda.synchronize()
                sec = a.elapsed_time(b) / 5 * 1e-3
                opt[name] = {"Gparam/s": round(n_p / sec / 1e9, 2), "GB/s": round(bpp * n_p / sec / 1e9, 1),
                             "frac_of_peak": round(bpp * n_p / sec / 1e9 / peak, 3), "params": n_p}
            extras["fused_optimizer_bf16_srf_k4"] = opt
            del w, m, v, g, lp
        except torch.OutOfMemoryError:
            extras["fused_optimizer_bf16_srf_k4"] = "skipped: out of memory"

    if rank == 0:
        # the oracle, as it stands, on a bounded sample of the same tensor (about 10-30 s of CPU work)
        sample = 1 << 22
        xh = x[:sample].cpu().numpy()
        threads = 1
        sec = time_oracle(xh, combos, offset, threads)
        cpu_baseline = {"value": sample * len(combos) / sec / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": "first 2^22 elements of the sweep tensor, all 48 (format, variant, k) combinations, once",
                        "host_cores_available": os.cpu_count()}
        # the same oracle on every host core (disjoint chunks, global index as offset), a larger sample
        all_threads = max(1, os.cpu_count() or 1)
        if all_threads > 1:
            big = min(n_local, (1 << 22) * min(all_threads, 8))
            xb = x[:big].cpu().numpy()
            sec_all = time_oracle(xb, combos, offset, all_threads)
            cpu_baseline["all_cores"] = {"value": big * len(combos) / sec_all / 1e9, "unit": UNIT, "cores": all_threads,
                                         "sample": "first %d elements, all 48 combinations, once" % big}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "u32", "data": "synthetic",
                "config": {"workload": "bandwidth sweep (2^28 fp32 per GPU -> bf16 and fp16; k in {1,2,3,4,6,8,13,16}; SRFF/SRF/SRC; seed 1234): 48 fbsr_round launches per step",
                           "elements_per_gpu": N_ELEMS, "launch_shapes": len(combos),
                           "l2": "inputs larger than L2 (1 GiB read, 512 MiB written per launch)"},
                "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches,
                "clocks": clocks, "extras": extras}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
