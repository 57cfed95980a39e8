"""N independent replicas of the decode step (the path does not shard: one GPU holds a whole layer's
cache and there is no exchange step, so there is no collective on the data path).  The only
cross-rank traffic is the measurement: a barrier around the timed region and the MAX of the ranks'
device times.  Works over NCCL (GPU ranks) and gloo (CPU tests)."""
from __future__ import annotations

import os


def init(backend: str, device=None):
    """Joins the process group named by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT.  Returns
    (rank, world) -- (0, 1) without a launcher."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world == 1:
        return 0, 1
    import torch.distributed as dist
    if not dist.is_initialized():
        if backend == "nccl" and device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(seconds: float, device="cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return seconds
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, seconds_this_rank: float, world: int, device="cpu") -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: every rank does
    the same work)."""
    return world * units_per_rank / max_over_ranks(seconds_this_rank, device)


def finish():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
