"""Multi-GPU plumbing of the benchmark: the path does not shard inside this library
(replicas only), so N ranks run N independent passes and only timing is exchanged."""
from __future__ import annotations


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar over the default process group (the value itself if
    torch.distributed is not initialised).  `device` is where the exchange tensor lives
    ("cuda" for NCCL, None/"cpu" for gloo)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world_size: int, slowest_ms: float) -> float:
    """Units per second of the whole job when every rank processes `units_per_rank`
    (weak scaling) and the slowest rank needs `slowest_ms`."""
    return world_size * units_per_rank / (slowest_ms * 1e-3)
