"""Multi-process plumbing of the benchmark: one process per GPU, each an independent replica of the
transfer (no data-path collective); only timings cross ranks."""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch


def rank_info() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment (1 process = defaults)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: Optional[torch.device] = None):
    """Join the process group when launched with WORLD_SIZE > 1; returns torch.distributed or None."""
    _, _, world = rank_info()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return dist


def barrier(dist, cuda: bool) -> None:
    if dist is not None:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(dist, value: float, device: torch.device) -> float:
    """The slowest rank's time: what a weak-scaling step costs."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(world: int, bytes_per_rank: int, ms: float) -> float:
    """Whole-job throughput of `world` replicas that each move bytes_per_rank in `ms`."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9
