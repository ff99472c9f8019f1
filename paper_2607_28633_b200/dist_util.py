"""The little that the data-parallel run needs from torch.distributed.

The path has no exchange step (every layer, request and page is independent), so ranks run
independent batches and only timing scalars cross ranks: the step time is the MAX over ranks,
the work is the SUM over ranks. NCCL on GPUs, gloo on CPU (tests)."""
from __future__ import annotations

import os

import torch


def env_rank_world():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None):
    """Initialises the default process group from the torchrun environment (MASTER_ADDR /
    MASTER_PORT / RANK / WORLD_SIZE), also for a world of one, so that the N = 1 leg of a
    scaling run goes through the same calls; returns the module, or None for a plain process."""
    rank, world, _ = env_rank_world()
    launched = "RANK" in os.environ and "MASTER_ADDR" in os.environ   # under torchrun
    if world <= 1 and not launched:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return dist


def _reduce(dist, x: float, op, device) -> float:
    if dist is None:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(dist, x: float, device=None) -> float:
    return _reduce(dist, x, None if dist is None else dist.ReduceOp.MAX, device)


def sum_over_ranks(dist, x: float, device=None) -> float:
    return _reduce(dist, x, None if dist is None else dist.ReduceOp.SUM, device)


def aggregate_throughput(dist, bytes_this_rank: float, ms_this_rank: float, device=None):
    """Whole-job GB/s = bytes of all ranks / the slowest rank's time. Returns (GB/s, ms)."""
    ms = max_over_ranks(dist, ms_this_rank, device)
    total = sum_over_ranks(dist, bytes_this_rank, device)
    return total / (ms * 1e-3) / 1e9, ms
