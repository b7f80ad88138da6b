"""Host-side logic for running the path on several GPUs of one node.

The path shards only by independent problems (signals / images of a batch, or
whole replicas of the workload): there is no data-path collective.  The only
communication is the timing protocol of the benchmark: a barrier on both sides
of the timed region and the maximum of the per-rank times.  Works with any
``torch.distributed`` backend (NCCL on GPUs, gloo on CPU for the tests).
"""


def split_range(total, rank, world):
    """Contiguous share [lo, hi) of ``total`` independent items for ``rank`` of ``world``.

    The first ``total % world`` ranks get one item more; shares are disjoint and cover the range.
    """
    if world < 1 or not (0 <= rank < world) or total < 0:
        raise ValueError("bad shard request: total=%r rank=%r world=%r" % (total, rank, world))
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value, world, device=None):
    """Maximum of a per-rank float over all ranks (the slowest rank defines the step time)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, world, device=None):
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank, seconds_this_rank, world, device=None):
    """Whole-job throughput: units processed by all ranks / the slowest rank's time."""
    total = sum_over_ranks(units_this_rank, world, device)
    slowest = max_over_ranks(seconds_this_rank, world, device)
    return total / slowest
