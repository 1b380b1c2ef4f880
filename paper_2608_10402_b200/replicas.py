"""Multi-GPU = independent replicas: a rollout data-parallel rank is its own token-budget pool with its own
KV cache, tasks are pinned to a rank and KV never moves between ranks (paper Sections 4.1, 4 end, 5.2), so
the path has no exchange step.  The only cross-rank work is bookkeeping for a benchmark: a barrier, the
MAX of the per-rank times and the SUM of the per-rank work."""
from __future__ import annotations


def rank_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own batch: a different, reproducible seed per rank."""
    return int(base_seed) + 7919 * int(rank)


def reduce_step_stats(times_ms, totals, world: int, dist=None, device="cpu"):
    """times_ms: list of per-rank times (reduced with MAX); totals: list of per-rank work counts (reduced
    with SUM).  Returns (times, totals) as Python floats, identical on every rank."""
    import torch
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    s = torch.tensor([float(x) for x in totals], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in s.tolist()]


def whole_job_rate(total_units: float, max_ms: float) -> float:
    """Units all ranks processed / the slowest rank's time (units per second)."""
    return total_units / (max_ms * 1e-3) if max_ms > 0 else 0.0
