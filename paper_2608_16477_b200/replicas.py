"""Host-side logic of the multi-GPU run: the path does not shard (one request's prefill is not an
independent-unit split), so N GPUs run N independent replicas, one request stream per rank, with no
data-path collective.  The only cross-rank traffic is the barrier around the timed region and the
max-over-ranks of the device time."""
from __future__ import annotations


def requests_of_rank(n_requests: int, world: int, rank: int) -> list[int]:
    """Round-robin partition of independent migration requests over ranks (request r runs on rank r % world)."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    return list(range(rank, n_requests, world))


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over all ranks (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: per-rank work is fixed)."""
    return world * units_per_rank / (slowest_ms * 1e-3)
