"""Host-side logic for running the rounding path on several GPUs (one process per GPU).

Elements are independent and every draw is keyed by the global element index, so the path
shards with no exchange step: rank r rounds elements [b[r], b[r+1]) of the flat tensor with
``offset = b[r]`` and the concatenation of the shards is bit-identical to a single call.
Only scalars cross ranks: the max of the step time and, when asked for, the sums of the
error statistics.  Nothing here touches the device; it is exercised on CPU with gloo.
"""
import math

def tile_elements(k_bits):
    """Elements per warp tile of the fast path (mirrors fbsr_tile_elements of the library)."""
    dpw = 32 // k_bits
    if dpw & (dpw - 1) == 0:
        return 1024
    rows = dpw // 2 if dpw % 2 == 0 else dpw
    if rows % 2:
        rows *= 2
    return rows * 256


TILE_ELEMENTS = {k: tile_elements(k) for k in range(1, 17)}
# every tile size divides this, so a shard boundary on this grid keeps all k on the fast path
SHARD_ALIGN = math.lcm(*TILE_ELEMENTS.values())

STAT_COUNTS = ("n_finite", "n_up", "n_nan", "n_inf", "n_sat")
STAT_SUMS = ("sum_e", "sum_e2", "sum_signed_e", "sum_abs_e")


def shard_bounds(n_total, world, align=SHARD_ALIGN):
    """world+1 non-decreasing boundaries; interior ones are multiples of `align` and the shards
    differ in size by at most `align` elements."""
    if world < 1 or n_total < 0 or align < 1:
        raise ValueError("bad arguments")
    blocks = -(-n_total // align)
    bounds = [min(n_total, (blocks * r // world) * align) for r in range(world)]
    bounds.append(n_total)
    return bounds


def my_shard(n_total, rank, world, align=SHARD_ALIGN):
    b = shard_bounds(n_total, world, align)
    return b[rank], b[rank + 1]


def max_over_ranks(value, dist=None, device="cpu"):
    """Max of a Python float over the process group (the value itself without a group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, dist=None, device="cpu"):
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64 if isinstance(value, float) else torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t.item()


def reduce_stats(stats, dist=None, device="cpu"):
    """Sum the per-shard error statistics (a dict as returned by fbsr_round_stats) over the group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return dict(stats)
    import torch
    counts = torch.tensor([int(stats[k]) for k in STAT_COUNTS], dtype=torch.int64, device=device)
    sums = torch.tensor([float(stats[k]) for k in STAT_SUMS], dtype=torch.float64, device=device)
    dist.all_reduce(counts, op=dist.ReduceOp.SUM)
    dist.all_reduce(sums, op=dist.ReduceOp.SUM)
    out = {k: int(v) for k, v in zip(STAT_COUNTS, counts.tolist())}
    out.update({k: float(v) for k, v in zip(STAT_SUMS, sums.tolist())})
    return out
