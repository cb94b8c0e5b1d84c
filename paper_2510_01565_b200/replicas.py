"""Multi-GPU deployment of the step: independent replicas, no data-path collective.

Requests of a packed batch never interact (block-diagonal attention), so N GPUs run N independent
batches.  The only cross-rank traffic is the timing protocol of the benchmark: a barrier on both
sides of the timed region and the maximum of the per-rank device times.
"""
from __future__ import annotations


def init_process_group(backend: str, device=None):
    """Joins the group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (torchrun's env)."""
    import torch.distributed as dist
    if dist.is_initialized():
        return dist
    kwargs = {}
    if device is not None and backend == "nccl":
        kwargs["device_id"] = device
    dist.init_process_group(backend, **kwargs)
    return dist


def max_over_ranks(ms: float, dist=None, device="cpu") -> float:
    """The slowest rank's time: what the whole job waited for."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world_size: int, ms_per_step: float) -> float:
    """Aggregate units per second of `world_size` replicas that each process `units_per_rank` per step."""
    return units_per_rank * world_size / (ms_per_step * 1e-3)
