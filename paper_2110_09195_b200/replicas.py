"""Host-side bookkeeping for running the conv stack on several GPUs.

Images are independent (Sec. 3: the layer is applied to every image alone), so a
multi-GPU run is a set of replicas: every rank owns a slice of the images, or a
whole batch of its own under weak scaling, and no activation or result crosses
ranks.  The only communication is the reduction of the ranks' timings, which
goes through whatever torch.distributed backend the job initialised (NCCL on
GPUs, gloo on CPU-only ranks).
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local_rank: int


def rank_info(env=None) -> RankInfo:
    """Rank layout from the launcher's environment (single process when unset)."""
    env = os.environ if env is None else env
    info = RankInfo(int(env.get("RANK", "0")), int(env.get("WORLD_SIZE", "1")), int(env.get("LOCAL_RANK", "0")))
    if info.world < 1 or not 0 <= info.rank < info.world:
        raise ValueError(f"inconsistent rank layout: rank {info.rank} of {info.world}")
    return info


def max_over_ranks(values, world: int, device=None):
    """Element-wise maximum of a short list of floats over all ranks (identity for one rank)."""
    vals = [float(v) for v in values]
    if world <= 1:
        return vals
    import torch
    import torch.distributed as dist

    t = torch.tensor(vals, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def sum_over_ranks(values, world: int, device=None):
    """Element-wise sum of a short list of numbers over all ranks."""
    vals = [float(v) for v in values]
    if world <= 1:
        return vals
    import torch
    import torch.distributed as dist

    t = torch.tensor(vals, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return [float(v) for v in t.cpu()]


def job_throughput(images_this_rank: int, ms_this_rank: float, world: int, device=None) -> tuple[float, float]:
    """Whole-job images per second and the time it is quoted on: all ranks' images
    over the slowest rank's time."""
    (ms,) = max_over_ranks([ms_this_rank], world, device)
    (images,) = sum_over_ranks([images_this_rank], world, device)
    if ms <= 0.0:
        raise ValueError("non-positive step time")
    return images / (ms * 1e-3), ms
