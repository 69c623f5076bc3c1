"""Multi-process plumbing of the benchmark: one process per GPU, replicas only.

Every probe of a table is independent of every other, so running on N GPUs means N processes
that each probe their own copy of the workload; nothing is exchanged in the data path.  What
the ranks do share is timing: a barrier on both sides of the timed region and the slowest
rank's time, from which the whole-job throughput is formed.
"""
import os

import torch
import torch.distributed as dist


def rank_info():
    """(rank, world size, local rank) from the torchrun environment; (0, 1, 0) without it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def barrier(world):
    if world > 1:
        dist.barrier()


def max_over_ranks(value, world, device="cpu"):
    """The largest `value` (a float, e.g. milliseconds) over all ranks, known to every rank."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank, world, slowest_ms):
    """Aggregate throughput (units per second) when every rank processed `units_per_rank` units
    and the slowest one took `slowest_ms` milliseconds (weak scaling: per-rank work is fixed)."""
    return units_per_rank * world / (slowest_ms * 1e-3)
