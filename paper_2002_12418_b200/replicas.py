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


def launch_plan(gpus: int, env) -> str:
    """How `bench.py --gpus N` gets its N ranks: "single" (N = 1), "env" (a launcher such as torchrun
    already started one process per rank: WORLD_SIZE is set), or "spawn" (N > 1 asked for on a plain
    command line: the benchmark starts the N local ranks itself)."""
    if "WORLD_SIZE" in env and int(env["WORLD_SIZE"]) >= 1 and "RANK" in env:
        return "env"
    return "single" if gpus <= 1 else "spawn"


def rank_environment(rank: int, world: int, port: int) -> dict:
    """Rendezvous variables of one locally spawned rank."""
    return {"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
            "MASTER_PORT": str(port)}
