"""Host-side helpers for running the BiGLA path on several GPUs, one process per GPU.

The (batch, head) units of Eq. 6 are independent, so the path shards by batch and needs no
data-path collective.  What remains is bookkeeping: which images a rank owns, and the job-wide
step time (the maximum over ranks of the device-measured time).
"""
from __future__ import annotations


def shard_range(n: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of n independent items owned by `rank` of `world` (sizes differ by <= 1)."""
    if world < 1 or not (0 <= rank < world) or n < 0:
        raise ValueError("need world >= 1, 0 <= rank < world, n >= 0")
    return range(n * rank // world, n * (rank + 1) // world)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Maximum of a per-rank scalar (e.g. an elapsed time in ms) over the process group; identity without one."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms_per_step_max: float, world: int) -> float:
    """Whole-job units per second when every rank processes units_per_rank per step (weak scaling)."""
    return world * units_per_rank / (ms_per_step_max * 1e-3)
