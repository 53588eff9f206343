"""Host-side plumbing for running the attention path on several GPUs of one node.

(batch, head) pairs -- and whole problems -- are independent, so the path shards with no exchange:
every rank gets a contiguous share of the problems and runs them on its own GPU; torch.distributed
is used only for the barrier around the timed region and for the maximum over ranks of the measured
time.  Nothing here touches the attention arithmetic.
"""
from __future__ import annotations


def shard(n_items: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of n_items for `rank` of `world` (sizes differ by at most one)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    lo = (n_items * rank) // world
    hi = (n_items * (rank + 1)) // world
    return range(lo, hi)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic problem a rank works on (one distinct problem per rank)."""
    return base_seed + rank


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Maximum of a per-rank scalar (the slowest rank's time); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist=None, device=None) -> float:
    """Sum of a per-rank scalar (work done by all ranks)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(work_this_rank: float, seconds_this_rank: float, dist=None, device=None) -> float:
    """Aggregate rate of the job: work of all ranks divided by the slowest rank's time."""
    total = sum_over_ranks(work_this_rank, dist, device)
    slowest = max_over_ranks(seconds_this_rank, dist, device)
    return total / slowest
