"""Multi-GPU plumbing of the benchmark: the path shards by images, every rank runs a full replica
on its own batch and there is no collective on the data path.  The only exchange is the timing:
the job's step time is the slowest rank's (MAX over ranks), the job's work the sum over ranks."""
from __future__ import annotations

import torch
import torch.distributed as dist


def job_throughput(local_ms_total: float, local_units: float, device="cpu") -> tuple:
    """(units per second of the whole job, max-over-ranks milliseconds).  Works without an
    initialised process group (single process)."""
    t = torch.tensor([float(local_ms_total)], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    ms = float(t.item())
    return float(u.item()) / (ms * 1e-3), ms


def shard_batch(total_images: int, rank: int, world: int) -> tuple:
    """Contiguous slice [start, stop) of a global batch for this rank (strong-scaling helper)."""
    base, extra = divmod(total_images, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)
