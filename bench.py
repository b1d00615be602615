#!/usr/bin/env python
"""Benchmark of the few-bit stochastic rounding path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload ("bandwidth sweep"): 2^28 binary32 elements per GPU, z ~ N(0,1) x 2^U(-20,20), seed 1234,
resident in HBM.  One step rounds the tensor to bfloat16 and to binary16 for every
k in {1,2,3,4,6,8,13,16} and every variant (SRFF, SRF, SRC): 48 fbsr_round launches.
Metric: elements rounded per second over the whole job (Gelem/s).

With --gpus N > 1 and no torchrun environment the script starts its own N ranks (one per GPU) through
torch.distributed.run on 127.0.0.1; under torchrun it uses the ranks it was given.  Every rank rounds its
own 2^28-element shard (weak scaling, no data-path collective); the N-rank run adds the statistics
all-reduce, a parameter-sharded Adam step (reduce-scatter, fused step, all-gather of the codes) and the
all-gather on its own.

Prints one JSON line (rank 0).  `--impl reference` times the scalar CPU oracle on a bounded
sample of the same workload.
"""
import argparse
import datetime
import json
import math
import os
import socket
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
NOMINAL_HBM_GBS = 8000.0        # the figure the >= 80 % targets are stated against


def sweep():
    return [(f, v, k) for f in FMT_LIST for v in VARIANT_LIST for k in K_LIST]


# DRAM traffic of one 2^28-element bf16 launch among back-to-back launches, from the ncu capture summarised
# in profiles/tile_kernel_round_traffic.txt (dram__bytes_read.sum + dram__bytes_write.sum of the second of two
# consecutive 2^28-element launches, so that the write-back of the previous launch's dirty lines is counted
# where it happens).  Valid only for the kernel sources it was taken from.
TRAFFIC_BYTES_PER_LAUNCH = 1073512704.0 + 537550592.0
TRAFFIC_KERNEL_SHA = "a39a07ba9d4b69ae"


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
    """Samples SM clocks and throttle reasons with nvidia-smi while timed regions run; summary() gives the
    median over everything sampled, window(t0, t1) over the samples taken between two time.time() values."""
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

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
        return self

    def _read(self):
        for line in self.proc.stdout:
            r = [t.strip() for t in line.split(",")]
            if len(r) < 10:
                continue
            try:
                stamp = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((stamp, float(r[2]), float(r[3]), r[6:10]))
            except ValueError:
                continue

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)

    def window(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [r for r in self.rows if (t0 is None or r[0] >= t0) and (t1 is None or r[0] <= t1)]
        sm = sorted(r[1] for r in rows)
        reasons = set()
        for r in rows:
            for name, val in zip(self.REASONS, r[3]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max((r[2] for r in rows), default=None),
                "reasons": sorted(reasons), "samples": len(sm)}


def time_oracle(work, n, threads):
    """Wall time of work(a, b) over [0, n) split into `threads` disjoint chunks on a thread pool."""
    import concurrent.futures
    cuts = [n * i // threads for i in range(threads + 1)]
    t0 = time.perf_counter()
    if threads == 1:
        work(0, n)
    else:
        with concurrent.futures.ThreadPoolExecutor(threads) as pool:
            list(pool.map(lambda i: work(cuts[i], cuts[i + 1]), range(threads)))
    return time.perf_counter() - t0


def oracle_sweep_seconds(x_host, combos, offset, threads):
    from oracle import capi
    capi.lib()

    def work(a, b):
        for fmt, variant, k in combos:
            capi.fbsr_round(x_host[a:b], fmt, variant, k, seed=SEED, offset=offset + a)

    return time_oracle(work, x_host.size, threads)


def run_reference(args, rank, world):
    """The scalar oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    from paper_2504_20634_b200 import workloads
    sample = 1 << 19
    x = workloads.bandwidth_sweep(sample, seed=SEED, device="cpu").numpy()
    combos = sweep()
    for _ in range(args.warmup):
        oracle_sweep_seconds(x[: sample // 8], combos[:6], 0, 1)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_sweep_seconds(x, combos, 0, 1)
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


# ---------------------------------------------------------------------------- starting the ranks
def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def respawn_command(argv, n):
    """The command that runs this script as n ranks on this node (one per GPU), rendezvous on 127.0.0.1."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)


def start_ranks_if_needed(args, argv):
    """`python bench.py --gpus N` without a torchrun environment: become N ranks."""
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        env = dict(os.environ)
        env.setdefault("NCCL_DEBUG", "INFO")          # the communicator's rank count shows in the log
        os.execvpe(sys.executable, respawn_command(argv, args.gpus), env)


def rendezvous_check(rank, world, local_rank):
    """Initialise the process group, all-reduce the ranks, report: the start-up path without any GPU work."""
    import torch.distributed as dist
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    if use_cuda:
        torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank) if use_cuda else torch.device("cpu")
    if world > 1:
        dist.init_process_group("nccl" if use_cuda else "gloo", **({"device_id": dev} if use_cuda else {}))
        t = torch.tensor([rank], dtype=torch.int64, device=dev)
        dist.all_reduce(t)
        total = int(t.item())
        dist.destroy_process_group()
    else:
        total = 0
    if rank == 0:
        print(json.dumps({"rendezvous": "ok" if total == world * (world - 1) // 2 else "mismatch", "n_gpus": world,
                          "backend": "nccl" if use_cuda else "gloo"}), flush=True)


# ---------------------------------------------------------------------------- timing helpers
def timed(fn, stream, min_seconds=1.0, warm=3):
    """Mean device time of fn(i) over a region of at least min_seconds (CUDA events on `stream`); returns
    (seconds per call, calls, host window of the timed region)."""
    for i in range(warm):
        fn(i)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for i in range(3):
        fn(warm + i)
    b.record(stream)
    torch.cuda.synchronize()
    est = max(a.elapsed_time(b) / 3 * 1e-3, 1e-7)
    iters = max(3, int(math.ceil(min_seconds / est)))
    t0 = time.time()
    a.record(stream)
    for i in range(iters):
        fn(warm + 3 + i)
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters * 1e-3, iters, (t0, time.time())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--skip-extras", action="store_true", help="skip the per-kernel table and the fused-optimizer timing")
    ap.add_argument("--rendezvous-check", action="store_true", help="start the ranks, all-reduce once, report and exit")
    args = ap.parse_args()

    if args.impl == "ours":
        start_ranks_if_needed(args, sys.argv[1:])
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.rendezvous_check:
        rendezvous_check(rank, world, local_rank)
        return

    import paper_2504_20634_b200 as fbsr            # raises if libfbsr.so is missing: no fallback
    from paper_2504_20634_b200 import sharding, workloads
    from paper_2504_20634_b200.sharded_optimizer import ShardedLowPrecisionAdam

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

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank).start()
    launches0 = fbsr.fbsr_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_host0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    t_host1 = time.time()
    launches = fbsr.fbsr_launch_count() - launches0
    ms = ev0.elapsed_time(ev1)
    ms = sharding.max_over_ranks(ms, dist, dev)
    launches = int(sharding.sum_over_ranks(int(launches), dist, dev))
    ms_per_step = ms / args.steps
    total_elems = float(N_ELEMS) * len(combos) * world
    value = total_elems / (ms_per_step * 1e-3) / 1e9

    # ---- the same step over a region of at least 3 s: what the power cap lets the kernels sustain
    sustained_steps = max(args.steps, int(math.ceil(3.0 / (ms_per_step * 1e-3))))
    barrier()
    s_host0 = time.time()
    ev0.record(stream)
    for _ in range(sustained_steps):
        step()
    ev1.record(stream)
    barrier()
    s_host1 = time.time()
    s_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev) / sustained_steps
    time.sleep(0.25)
    clocks = sampler.window(t_host0, t_host1)
    if not clocks.get("samples"):
        clocks = sampler.window(t_host0 - 0.2, s_host1)        # a timed region shorter than the sampling period
    sustained = {"steps": sustained_steps, "seconds": s_ms * sustained_steps * 1e-3, "ms_per_step": s_ms,
                 "value": total_elems / (s_ms * 1e-3) / 1e9, "unit": UNIT,
                 "GB/s": BYTES_PER_ELEM * n_local * len(combos) / (s_ms * 1e-3) / 1e9,
                 "clocks": sampler.window(s_host0, s_host1)}

    # ---- roofline of the tiled rounding kernel: all 48 launches move 6 B/element
    peak, peak_kind = measured_peak_gbs()
    sec_per_launch = ms_per_step * 1e-3 / len(combos)
    achieved = BYTES_PER_ELEM * n_local / sec_per_launch / 1e9
    traffic = TRAFFIC_BYTES_PER_LAUNCH if kernel_source_sha() == TRAFFIC_KERNEL_SHA else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic,
                "peak_source": peak_kind + " copy bandwidth (a plain copy's rate on this pool, not a ceiling: a kernel "
                                           "that streams 4 B in and 2 B out can pass it)",
                "kernel": "fbsr::tile_kernel<RoundOp, fmt, variant, k> (average over the 48 launches of a step)",
                "algorithmic_bytes_per_launch": BYTES_PER_ELEM * n_local,
                "frac_of_8TBps_algorithmic": achieved / NOMINAL_HBM_GBS,
                "achieved_traffic": traffic / sec_per_launch / 1e9 if traffic else None,
                "frac_of_8TBps_traffic": traffic / sec_per_launch / 1e9 / NOMINAL_HBM_GBS if traffic else None,
                "target_judged_on": "algorithmic bytes over 8 TB/s (>= 0.80); in back-to-back launches, where the previous "
                                    "launch's dirty L2 lines are written back during the next one, the measured traffic "
                                    "per launch is 1.0003 x the algorithmic bytes, so both fractions agree"}

    # ---- end to end through the host-buffer entry point on the whole 2^28-element tensor (pinned host
    # memory, copies inside the timed region, the last code read on the host every step)
    e2e = None
    n_e2e = n_local
    src_h = torch.empty(n_e2e, dtype=torch.float32).pin_memory()
    src_h.copy_(x[:n_e2e])
    dst_h = torch.empty(n_e2e, dtype=torch.uint16).pin_memory()
    ws = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def e2e_step():
        for fmt, variant, k in combos:
            fbsr.fbsr_round_host(src_h, dst_h, fmt, variant, k, SEED, offset, 1.0, ws)
        stream.synchronize()
        return int(dst_h[-1])          # the step's result is read on the host

    e2e_step()
    barrier()
    e2e_steps = max(1, min(args.steps, 3))
    ev0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    ev1.record(stream)
    barrier()
    e_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    e_val = float(n_e2e) * len(combos) * e2e_steps * world / (e_ms * 1e-3) / 1e9
    e2e = {"value": e_val, "unit": UNIT, "h2d_bytes_per_step": 4 * n_e2e * len(combos),
           "d2h_bytes_per_step": 2 * n_e2e * len(combos),
           "note": "fbsr_round_host on the whole 2^28-element tensor in pinned host memory, 48 calls per step, %d steps" % e2e_steps}
    del src_h, dst_h, ws

    # ---- legs that only exist on several ranks (they also run, without collectives, on one)
    multi = {}
    # error statistics of the shard, then one all-reduce of the nine numbers
    ws_stats = torch.empty(fbsr.fbsr_stats_workspace_bytes(), dtype=torch.uint8, device=dev)
    total_dev = torch.empty(72, dtype=torch.uint8, device=dev)
    fbsr.fbsr_round_stats(x, "bf16", "srf", 2, seed=SEED, offset=offset, out=out, workspace=ws_stats, total=total_dev,
                          read_back=False)
    barrier()
    ev0.record(stream)
    fbsr.fbsr_round_stats(x, "bf16", "srf", 2, seed=SEED, offset=offset, out=out, workspace=ws_stats, total=total_dev,
                          read_back=False)
    ev1.record(stream)
    stats_all = sharding.reduce_stats(fbsr.stats_from_bytes(total_dev), dist, dev)
    barrier()
    st_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev)
    multi["round_stats_bf16_srf_k2"] = {"Gelem/s": float(n_local) * world / (st_ms * 1e-3) / 1e9,
                                        "bias_ulps": stats_all["sum_e"] / max(stats_all["n_finite"], 1),
                                        "n_finite": stats_all["n_finite"]}
    del ws_stats, total_dev
    # parameter-sharded fused Adam: every rank owns 2^27 parameters' master weights and moments
    n_params = world * (1 << 27)
    opt = ShardedLowPrecisionAdam(n_params, fmt="bf16", variant="srf", k_bits=4, seed=SEED, device=dev)
    opt.load_master(workloads.optimizer_state(opt.n_own, seed=99 + rank, device=dev)[0])
    gbuf = opt.grad_buffer()
    gbuf.normal_(0.0, 1e-3)

    def sharded_step():
        opt.step(opt.reduce_scatter_grad(), wait=False)

    for _ in range(3):
        sharded_step()
    opt.wait_gather()
    barrier()
    ev0.record(stream)
    for _ in range(10):
        sharded_step()
    opt.wait_gather()
    ev1.record(stream)
    barrier()
    sh_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev) / 10
    multi["sharded_adam_bf16_srf_k4"] = {"params": n_params, "Gparam/s": n_params / (sh_ms * 1e-3) / 1e9,
                                         "ms_per_step": sh_ms,
                                         "note": "gradient reduce-scatter, fused step on the shard, all-gather of the bf16 codes"}
    if dist is not None:
        own = opt._own_slice().view(torch.uint8)
        full = opt.lp_padded.view(torch.uint8)
        for _ in range(3):
            dist.all_gather_into_tensor(full, own)
        barrier()
        ev0.record(stream)
        for _ in range(10):
            dist.all_gather_into_tensor(full, own)
        ev1.record(stream)
        barrier()
        ag_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist, dev) / 10
        multi["all_gather_bf16_codes"] = {"bytes_per_rank": own.numel(), "ms": ag_ms,
                                          "GB/s_received_per_rank": own.numel() * (world - 1) / (ag_ms * 1e-3) / 1e9}
    del opt, gbuf
    torch.cuda.empty_cache()

    extras = {}
    if rank == 0 and world == 1 and not args.skip_extras:
        extras = run_extras(fbsr, workloads, x, out, offset, n_local, dev, stream, peak, sampler)
    sampler.stop()

    cpu_baseline = None
    if rank == 0:
        cpu_baseline = run_cpu_baselines(workloads, x, combos, offset, n_local, quick=args.skip_extras)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "u32", "data": "synthetic",
                "config": {"workload": "bandwidth sweep (2^28 fp32 per GPU -> bf16 and fp16; k in {1,2,3,4,6,8,13,16}; SRFF/SRF/SRC; seed 1234): 48 fbsr_round launches per step",
                           "elements_per_gpu": N_ELEMS, "launch_shapes": len(combos),
                           "l2": "inputs larger than L2 (1 GiB read, 512 MiB written per launch)"},
                "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches,
                "clocks": clocks, "sustained": sustained, "multi_rank_legs": multi, "extras": extras}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_extras(fbsr, workloads, x, out, offset, n_local, dev, stream, peak, sampler):
    """Per-kernel figures, each over a timed region of at least one second, with the median SM clock of that
    region.  Not part of the headline step."""
    extras = {}

    def leg(fn, nbytes, min_seconds=1.0):
        sec, iters, (t0, t1) = timed(fn, stream, min_seconds)
        w = sampler.window(t0, t1)
        return {"GB/s": round(nbytes / sec / 1e9, 1), "calls": iters, "sm_mhz": w.get("sm_mhz")}, sec

    # every launch shape of the sweep
    table = {}
    for fmt, variant, k in sweep():
        r, _ = leg(lambda i: fbsr.fbsr_round(x, fmt, variant, k, seed=SEED, offset=offset, out=out), BYTES_PER_ELEM * n_local)
        table["%s/%s/k%d" % (fmt, variant, k)] = r
    extras["round_GBps"] = table
    # a source that starts 4 bytes off a 32-byte boundary, and codes 2 bytes off a 16-byte one (a slice of a larger buffer)
    xm = workloads.bandwidth_sweep(n_local + 8, seed=SEED, device=dev)
    om = torch.empty(n_local + 8, dtype=torch.uint16, device=dev)
    r, _ = leg(lambda i: fbsr.fbsr_round(xm[1:n_local + 1], "bf16", "srf", 4, seed=SEED, out=out), BYTES_PER_ELEM * n_local)
    extras["round_misaligned_src_GBps"] = r
    r, _ = leg(lambda i: fbsr.fbsr_round(xm[1:n_local + 1], "bf16", "srf", 4, seed=SEED, out=om[1:n_local + 1]), BYTES_PER_ELEM * n_local)
    extras["round_misaligned_src_and_dst_GBps"] = r
    del xm, om
    # the paper-literal overflow option on the sweep data (about 10 % of the fp16 elements overflow)
    t = {}
    for fmt in ("bf16", "fp16"):
        r, _ = leg(lambda i: fbsr.fbsr_round(x, fmt + "+ieee", "srf", 4, seed=SEED, offset=offset, out=out), BYTES_PER_ELEM * n_local)
        t["%s/srf/k4" % fmt] = r
    extras["round_ieee_overflow_GBps"] = t
    # fp8 leg of the metric (5 B/element): the 4096 x 32768 activation workload
    t8 = {}
    out8 = torch.empty(1 << 27, dtype=torch.uint8, device=dev)
    for fmt in ("e4m3", "e5m2", "b8p4"):
        xa, scale = workloads.fp8_activations(fmt, device=dev)
        for k in (2, 4, 8):
            r, _ = leg(lambda i: fbsr.fbsr_round(xa, fmt, "srf", k, seed=7, scale=scale, out=out8), 5.0 * (1 << 27))
            t8["%s/srf/k%d" % (fmt, k)] = r
        r, _ = leg(lambda i: fbsr.fbsr_round(xa, fmt, "src", 4, seed=7, scale=scale, out=out8), 5.0 * (1 << 27))
        t8["%s/src/k4" % fmt] = r
        del xa
    extras["round_fp8_GBps"] = t8
    # rounding with the fused error statistics (the C-ABI call alone: the totals stay on the device)
    ts = {}
    ws_stats = torch.empty(fbsr.fbsr_stats_workspace_bytes(), dtype=torch.uint8, device=dev)
    total_dev = torch.empty(72, dtype=torch.uint8, device=dev)
    for fmt, variant, k in (("bf16", "srf", 2), ("bf16", "src", 3), ("fp16", "srf", 3)):
        r, _ = leg(lambda i: fbsr.fbsr_round_stats(x, fmt, variant, k, seed=7, out=out, workspace=ws_stats, total=total_dev,
                                                   read_back=False), 6.0 * n_local)
        ts["%s/%s/k%d sweep" % (fmt, variant, k)] = r
    for fmt, variant, k in (("e4m3", "srf", 3), ("e5m2", "src", 4), ("b8p4", "src", 3)):
        xa, scale = workloads.fp8_activations(fmt, device=dev)
        r, _ = leg(lambda i: fbsr.fbsr_round_stats(xa, fmt, variant, k, seed=7, scale=scale, out=out8, workspace=ws_stats,
                                                   total=total_dev, read_back=False), 5.0 * (1 << 27))
        ts["%s/%s/k%d activations" % (fmt, variant, k)] = r
        del xa
    x8 = x[: 1 << 27]
    r, _ = leg(lambda i: fbsr.fbsr_round_stats(x8, "e4m3", "srf", 3, seed=7, scale=2.0 ** -10, out=out8, workspace=ws_stats,
                                               total=total_dev, read_back=False), 5.0 * (1 << 27))
    ts["e4m3/srf/k3 sweep x 2^-10 (half the elements below the subnormal range)"] = r
    extras["round_stats_GBps"] = ts
    del ws_stats, total_dev
    # a format described at run time: float8_e4m3fnuz = (8, 4, 8; 240), 5 B/element
    desc = fbsr.format_desc(8, 4, 8, 0x7F, None, 0x80, True)
    td = {}
    for k in (3, 8):
        r, _ = leg(lambda i: fbsr.fbsr_round_desc(x8, desc, "srf", k, seed=7, scale=2.0 ** -10, out=out8), 5.0 * (1 << 27))
        td["(8,4,8;240)/srf/k%d" % k] = r
    extras["round_desc_GBps"] = td
    # block-scaled rounding (blocks of 32, fused block maximum)
    scales = torch.empty(n_local // 32, dtype=torch.uint8, device=dev)
    w8 = torch.empty(n_local, dtype=torch.uint8, device=dev)
    r, _ = leg(lambda i: fbsr.fbsr_round_mx(x, "e4m3", "srf", 4, seed=SEED, out=w8, scales=scales), (5.0 + 1.0 / 32) * n_local)
    extras["round_mx_e4m3_srf_k4_GBps"] = r
    # supplied random bits
    dpw = 32 // 4
    words = torch.randint(0, 2 ** 31, (n_local // dpw,), device=dev, dtype=torch.int32).view(torch.uint32)
    r, _ = leg(lambda i: fbsr.fbsr_round_bits(x, "bf16", "srf", 4, words, out=out), (6.0 + 4.0 / dpw) * n_local)
    extras["round_bits_bf16_srf_k4_GBps"] = r
    del x8, out8, scales, words
    # 16-bit sources into 8-bit formats (3 B/element) and the 16-bit-sum weight update (4 B/element)
    codes16 = workloads.lp_sweep(n_local, "bf16", device=dev)
    tlp = {}
    for fmt in ("e4m3", "e5m2", "b8p4"):
        for variant in VARIANT_LIST:
            r, _ = leg(lambda i: fbsr.fbsr_round_lp(codes16, "bf16", fmt, variant, 3, seed=SEED, out=w8), 3.0 * n_local)
            tlp["bf16->%s/%s/k3" % (fmt, variant)] = r
    extras["round_lp_GBps"] = tlp
    upd = (torch.randn(n_local, device=dev) * 0.01).to(torch.bfloat16).view(torch.uint16)
    for wf in ("e4m3", "b8p4"):
        fbsr.fbsr_round_lp(codes16, "bf16", wf, "rtne", 1, seed=0, out=w8)
        r, _ = leg(lambda i: fbsr.fbsr_qat_update(w8, upd, wf, "bf16", "src", 3, seed=1 + i), 4.0 * n_local)
        extras["qat_update_%s_bf16_src_k3_GBps" % wf] = r
    # one whole iteration of Algorithm 1, fused (20 B/parameter): Binary8P4 weights, bf16 gradients, 3 random bits
    m_ = torch.zeros(n_local, device=dev)
    v_ = torch.zeros(n_local, device=dev)
    r, sec = leg(lambda i: fbsr.fbsr_qat_adamw_step(w8, upd, m_, v_, "b8p4", "bf16", "src", 3, 1 + i, 0, 1e-3, 0.9, 0.95, 1e-8,
                                                    0.1, 1 + i), 20.0 * n_local)
    r["Gparam/s"] = round(n_local / sec / 1e9, 2)
    extras["qat_adamw_step_b8p4_bf16_src_k3"] = r
    # accumulation into stored bf16 weights (8 B/element)
    wacc = workloads.accumulation_weights(n_local, device=dev)
    r, _ = leg(lambda i: fbsr.fbsr_accumulate(wacc, m_, "bf16", "srf", 4, seed=1 + i), 8.0 * n_local)
    extras["accumulate_bf16_srf_k4_GBps"] = r
    del codes16, w8, upd, m_, v_, wacc
    torch.cuda.empty_cache()
    # fused optimizer step on the 32-block parameter list (22 B/param SGD-momentum, 30 B/param Adam)
    try:
        n_p = workloads.optimizer_param_count(32)
        w, m, v = workloads.optimizer_state(n_p, device=dev)
        g = workloads.optimizer_grad(n_p, 1, device=dev)
        lp = torch.empty(n_p, dtype=torch.uint16, device=dev)
        opt = {}
        for name, fn, bpp in (("sgd_momentum", lambda s: fbsr.fbsr_sgd_update(w, g, m, "bf16", "srf", 4, SEED + s, 0, 1e-4, 0.9, out=lp), 22.0),
                              ("adam", lambda s: fbsr.fbsr_adam_update(w, g, m, v, "bf16", "srf", 4, SEED + s, 0, 1e-4, 0.9, 0.999, 1e-8, s + 1, out=lp), 30.0)):
            r, sec = leg(fn, bpp * n_p)
            r.update({"Gparam/s": round(n_p / sec / 1e9, 2), "frac_of_8TBps": round(bpp * n_p / sec / 1e9 / NOMINAL_HBM_GBS, 3),
                      "frac_of_measured_copy": round(bpp * n_p / sec / 1e9 / peak, 3), "params": n_p})
            opt[name] = r
        extras["fused_optimizer_bf16_srf_k4"] = opt
        del w, m, v, g, lp
    except torch.OutOfMemoryError:
        extras["fused_optimizer_bf16_srf_k4"] = "skipped: out of memory"
    return extras


def run_cpu_baselines(workloads, x, combos, offset, n_local, quick=False):
    """The oracle, as it stands, on bounded samples of each configuration: one thread and every host core
    (disjoint chunks, the global index as offset)."""
    import numpy as np
    from oracle import capi
    capi.lib()
    cores = max(1, os.cpu_count() or 1)
    sample = 1 << 22
    xh = x[:sample].cpu().numpy()
    sec = oracle_sweep_seconds(xh, combos, offset, 1)
    base = {"value": sample * len(combos) / sec / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "first 2^22 elements of the sweep tensor, all 48 (format, variant, k) combinations, once",
            "host_cores_available": cores}
    if cores > 1:
        big = min(n_local, (1 << 22) * min(cores, 8))
        xb = x[:big].cpu().numpy()
        sec_all = oracle_sweep_seconds(xb, combos, offset, cores)
        base["all_cores"] = {"value": big * len(combos) / sec_all / 1e9, "unit": UNIT, "cores": cores,
                             "sample": "first %d elements, all 48 combinations, once" % big}
    if quick:
        return base
    per = {}
    # fp8 activations: both formats, k in {2, 4, 8}, every variant
    n8 = 1 << 21
    xa, scale = workloads.fp8_activations("e4m3", rows=n8 // 32768, cols=32768, device="cpu")
    xa = xa.numpy()
    c8 = [(f, v, k) for f in ("e4m3", "e5m2") for v in VARIANT_LIST for k in (2, 4, 8)]

    def fp8(a, b):
        for f, v, k in c8:
            capi.fbsr_round(xa[a:b], f, v, k, seed=7, offset=a, scale=scale)

    per["fp8_activations"] = {"unit": "Gelem/s", "one_core": n8 * len(c8) / time_oracle(fp8, n8, 1) / 1e9}
    # fused optimizer steps and accumulation
    n4 = 1 << 22
    w0, m0, v0 = (t.numpy() for t in workloads.optimizer_state(n4, device="cpu"))
    g0 = workloads.optimizer_grad(n4, 1, device="cpu").numpy()
    wl = workloads.accumulation_weights(n4, device="cpu").view(torch.int16).numpy().view(np.uint16)

    def sgd(a, b):
        capi.sgd_update(w0[a:b], g0[a:b], m0[a:b], "bf16", "srf", 4, seed=1, offset=a, lr=1e-4, mu=0.9)

    def adam(a, b):
        capi.adam_update(w0[a:b], g0[a:b], m0[a:b], v0[a:b], "bf16", "srf", 4, seed=1, offset=a, lr=1e-4, beta1=0.9,
                         beta2=0.999, eps=1e-8, step=1)

    def accum(a, b):
        capi.accumulate(wl[a:b], g0[a:b], "bf16", "srf", 4, seed=1, offset=a)

    for name, fn, unit in (("sgd_momentum", sgd, "Gparam/s"), ("adam", adam, "Gparam/s"), ("accumulate", accum, "Gelem/s")):
        per[name] = {"unit": unit, "one_core": n4 / time_oracle(fn, n4, 1) / 1e9}
    if cores > 1:
        per["fp8_activations"]["all_cores"] = n8 * len(c8) / time_oracle(fp8, n8, cores) / 1e9
        for name, fn in (("sgd_momentum", sgd), ("adam", adam), ("accumulate", accum)):
            per[name]["all_cores"] = n4 / time_oracle(fn, n4, cores) / 1e9
    per["cores"] = cores
    per["sample"] = "fp8: 2^21 activations x 18 (format, variant, k); optimizer and accumulation: 2^22 parameters, one step"
    base["per_config"] = per
    return base


if __name__ == "__main__":
    main()
