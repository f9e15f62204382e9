"""Multi-GPU bookkeeping of the re-layout: replicas only.

On one device per model the path has no exchange step, so N GPUs run N independent
replicas of the same scale step (one process per GPU).  The only things ranks share
are a barrier before the timed region and the reduction of their step times: the
job's time is the slowest rank's, its throughput the bytes all replicas moved over
that time.  No collective touches the data path.
"""
from __future__ import annotations


def job_time_ms(local_ms: float, dist=None, device=None) -> float:
    """Max over ranks of a locally measured duration (all ranks must call it).

    dist: an initialised torch.distributed module, or None for a single process.
    device: where the reduction tensor lives ("cuda" for nccl, None/"cpu" for gloo).
    """
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms)
    import torch
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput_gbs(bytes_moved_per_replica: int, world_size: int, step_ms: float) -> float:
    """Whole-job reshard GB/s: every byte of the new layout is read once and written once
    (2 x bytes moved), summed over the replicas, over the slowest rank's step time."""
    if step_ms <= 0:
        raise ValueError("step time must be positive")
    return world_size * 2.0 * bytes_moved_per_replica / (step_ms * 1e-3) / 1e9
