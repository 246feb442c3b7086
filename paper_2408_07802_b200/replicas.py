"""Host-side logic of the multi-GPU mode: independent replicas, no data-path collective.

The Kraken path as built here runs whole on one GPU, so N GPUs serve N independent request
batches.  The only cross-rank steps are the barrier around the timed region and the max over
ranks of the measured time; both go through torch.distributed (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def rank_env() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def token_seed(rank: int, base: int = 1) -> int:
    """Every replica serves its own request stream: distinct seeded tokens per rank."""
    return base + rank


def init_process_group(backend: str, device: Optional[torch.device] = None):
    import torch.distributed as dist
    if dist.is_initialized():
        return dist
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend, **kw)
    return dist


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def whole_job_throughput(units_per_rank: float, ms_max_over_ranks: float, world: int) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / (ms_max_over_ranks * 1e-3)
