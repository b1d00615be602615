"""The multi-GPU path on CPU: two gloo ranks round their shards (the oracle stands in for the
device kernels, which need a GPU) and the host logic -- shard boundaries, offsets, reduction of the
statistics and of the step time -- must reproduce the single-call result exactly."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2504_20634_b200 import sharding


def test_shard_bounds_properties():
    for n, world in ((0, 1), (1, 4), (61440, 2), (2 ** 28, 1), (2 ** 29, 2), (8 * 2 ** 28, 8), (10 ** 6 + 7, 3)):
        b = sharding.shard_bounds(n, world)
        assert len(b) == world + 1 and b[0] == 0 and b[-1] == n
        assert all(x <= y for x, y in zip(b[:-1], b[1:]))
        assert all(x % sharding.SHARD_ALIGN == 0 for x in b[1:-1])
        sizes = [y - x for x, y in zip(b[:-1], b[1:])]
        if n >= world * sharding.SHARD_ALIGN:
            assert max(sizes) - min(sizes) <= sharding.SHARD_ALIGN
    for k in range(1, 17):
        assert sharding.SHARD_ALIGN % sharding.TILE_ELEMENTS[k] == 0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_total, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import capi
        from paper_2504_20634_b200 import workloads
        x = workloads.bandwidth_sweep(n_total, seed=1234, device="cpu").numpy()       # same tensor on every rank
        lo, hi = sharding.my_shard(n_total, rank, world, align=sharding.TILE_ELEMENTS[3])
        codes, st, _, _ = capi.fbsr_round_stats(x[lo:hi], "fp16", "src", 3, seed=1234, offset=lo, scale=0.5)
        total = sharding.reduce_stats(st, dist)
        slowest = sharding.max_over_ranks(1.0 + rank, dist)
        n_sum = sharding.sum_over_ranks(hi - lo, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, codes))
        if rank == 0:
            whole, wst, _, _ = capi.fbsr_round_stats(x, "fp16", "src", 3, seed=1234, offset=0, scale=0.5)
            cat = np.concatenate([g[2] for g in sorted(gathered, key=lambda g: g[0])])
            ok = np.array_equal(cat, whole) and n_sum == n_total and slowest == float(world)
            for key in sharding.STAT_COUNTS:
                ok = ok and total[key] == wst[key]
            for key in sharding.STAT_SUMS:
                ok = ok and abs(total[key] - wst[key]) <= 1e-9 * max(abs(wst[key]), 1.0)
            with open(os.path.join(out_dir, "result"), "w") as fh:
                fh.write("ok" if ok else "mismatch")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_rounding_equals_single_call(tmp_path, world):
    n_total = 5 * sharding.TILE_ELEMENTS[3] + 123
    mp.spawn(_worker, args=(world, _free_port(), n_total, str(tmp_path)), nprocs=world, join=True)
    assert open(tmp_path / "result").read() == "ok"
