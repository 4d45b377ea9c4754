"""Multi-GPU plumbing of the benchmark: the path does not shard (the paper is single-GPU and the step has no exchange),
so N GPUs run N independent replicas of the step.  The only cross-rank traffic is a barrier around the timed region
and the maximum of the per-rank step times; the job's throughput is the units all ranks processed over that time."""
from __future__ import annotations


def max_over_ranks(ms_local: float, world: int, device="cpu") -> float:
    """Slowest rank's time (collective: every rank of the default process group must call it)."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job units per second of `world` replicas that each process `units_per_rank` units per step."""
    return world * units_per_rank / (ms_per_step * 1e-3)
