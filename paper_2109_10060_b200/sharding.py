"""Batch sharding across GPUs.  The path is independent per sample (every input runs the route its own
gate picks), so ranks take contiguous batch shards with replicated weights and exchange nothing on the
data path; the only collectives are for reporting (routing histogram, step time)."""
from __future__ import annotations


def shard_range(B: int, rank: int, world: int):
    """Contiguous shard [lo, hi) of a batch of B samples for `rank` of `world` (sizes differ by at most 1)."""
    if world < 1 or not 0 <= rank < world or B < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def reduce_histogram(counts, dist=None):
    """Sum of the per-rank routing histograms (a tensor of T integers); identity without a process group."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(counts, op=dist.ReduceOp.SUM)
    return counts


def max_over_ranks(value, dist=None):
    """Largest value of a one-element tensor over all ranks (step time of the slowest rank)."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(value, op=dist.ReduceOp.MAX)
    return value
