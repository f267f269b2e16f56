"""Caller-side sharding helpers for running the library on several GPUs.

The method needs no exchange between devices: every element of C depends on one row of A and
one column of B, a convolution's output image n depends on input image n only, and a skinny
GEMM splits over weight rows.  So multi-GPU use is one process per GPU, each calling the
library on its own shard; these helpers only do the bookkeeping (index ranges, and the
max-over-ranks time / aggregate throughput a benchmark reports).  No data-path collective.
"""
from __future__ import annotations


def shard_range(total: int, rank: int, world: int, multiple: int = 1):
    """Half-open range [lo, hi) of `total` units owned by `rank`; boundaries are multiples of
    `multiple` (e.g. 128 rows, so shards start on tile boundaries), block counts differ by at most
    one (the last block may be partial), and the `world` ranges tile [0, total) exactly."""
    if world <= 0 or not (0 <= rank < world) or total < 0 or multiple <= 0:
        raise ValueError("bad shard request")
    blocks = -(-total // multiple)
    base, extra = divmod(blocks, world)
    lo_b = rank * base + min(rank, extra)
    hi_b = lo_b + base + (1 if rank < extra else 0)
    return min(lo_b * multiple, total), min(hi_b * multiple, total)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Maximum of a per-rank scalar (elapsed time); identity without a process group."""
    if dist is None or not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, elapsed_s_per_rank: float, world: int, dist=None, device=None) -> float:
    """Whole-job throughput for weak scaling: every rank processed `units_per_rank`, the job took
    as long as its slowest rank."""
    worst = max_over_ranks(elapsed_s_per_rank, dist, device)
    return world * units_per_rank / worst
