"""Host-side logic of the multi-GPU benchmark: images are independent, so N ranks run N
replicas of the path on their own batches (weak scaling) and exchange nothing but timing.
Kept free of CUDA so that it can be exercised with the gloo backend on CPU."""
from __future__ import annotations


def rank_seed_offset(rank: int) -> int:
    """Offset added to a layer's seed on `rank`, so that every rank draws its own batch."""
    return 10000 * rank


def max_over_ranks(dist, value: float, device=None) -> float:
    """The largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(flops_per_rank_step: float, steps: int, world: int, slowest_ms: float) -> float:
    """Aggregate TFLOP/s of `world` replicas that each did `steps` steps in at most `slowest_ms`."""
    return world * flops_per_rank_step * steps / (slowest_ms * 1e-3) / 1e12
