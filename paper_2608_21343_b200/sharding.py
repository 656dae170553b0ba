"""How a job is spread over several GPUs: streams are independent, so each rank decodes its own
streams and nothing crosses ranks on the data path.  The only collective is the reduction of the
timing (the job is as slow as its slowest rank)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_streams(rank: int, streams_per_rank: int) -> list:
    """Weak scaling: every rank gets its own `streams_per_rank` stream ids, disjoint across ranks."""
    return [rank * streams_per_rank + i for i in range(streams_per_rank)]


def job_throughput(frames_this_rank: int, ms_this_rank: float, device=None) -> dict:
    """Whole-job frames/s: frames of all ranks over the slowest rank's time (max over ranks)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return dict(ms=ms_this_rank, frames=frames_this_rank, value=frames_this_rank / (ms_this_rank * 1e-3), world=1)
    t = torch.tensor([ms_this_rank], dtype=torch.float64, device=device)
    f = torch.tensor([float(frames_this_rank)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return dict(ms=float(t.item()), frames=int(f.item()), value=float(f.item()) / (float(t.item()) * 1e-3),
                world=dist.get_world_size())
