"""Host-side plumbing for running one replica of the path per GPU (no collective on the data path).

Lowered rows are independent, so several GPUs split the batch: each rank holds its own images,
weights, mask and kept-row list and writes its own slice of the output.  The only cross-rank
steps are the barrier around a timed region and the maximum of the ranks' elapsed times.
"""
from __future__ import annotations

from typing import Tuple


def shard_batch(Nb: int, rank: int, world: int) -> Tuple[int, int]:
    """Images [lo, hi) of a batch of Nb that rank `rank` of `world` processes (strong scaling)."""
    if not (0 <= rank < world) or Nb < 0:
        raise ValueError("bad rank/world/batch")
    base, extra = divmod(Nb, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (the slowest rank's elapsed time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, ms_per_step_max: float, world: int) -> float:
    """Aggregate throughput when every rank processes `units_per_rank` per step (weak scaling)
    and the step takes the slowest rank's time."""
    return world * units_per_rank / (ms_per_step_max * 1e-3)
