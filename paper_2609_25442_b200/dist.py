"""Multi-process plumbing: one process per GPU.

The benchmark runs independent replicas of the transfer (no data-path collective; only timings cross
processes).  The rank-sharded transfer - virtual trainer and rollout ranks spread over the processes,
each packing its own senders' slabs, one exchange of (receiver, sender) bucket regions, each assembling
its own receivers' parameters (Section 3.2: per-worker packing and assembly around the receive stage) -
is stated here as well; its partition and exchange logic is exercised with gloo processes on the CPU."""
from __future__ import annotations

import os
from typing import List, Optional, Sequence, Tuple

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


def block_owner(n_virtual_ranks: int, world: int) -> List[int]:
    """Process that owns each virtual rank: contiguous blocks, as even as possible."""
    return [v * world // n_virtual_ranks for v in range(n_virtual_ranks)]


def exchange_regions(dist, bucket: torch.Tensor, regions, trainer_owner: Sequence[int],
                     rollout_owner: Sequence[int], me: int) -> int:
    """The receive stage for one round: every (receiver, sender) region of `bucket` (a flat uint8 tensor
    laid out as the plan says, on the CPU for gloo or on this process's GPU for NCCL) travels from the
    process that owns the sender to the process that owns the receiver, to the same offset there.
    Regions whose two owners coincide stay where they are.  Sizes are fixed by the plan, so both sides
    post matching point-to-point operations in region order (an all-to-all-v written out).  Returns the
    bytes this process sent."""
    ops, sent = [], 0
    for g in regions:
        a, b = trainer_owner[int(g["sender"])], rollout_owner[int(g["receiver"])]
        if a == b or int(g["bytes"]) == 0:
            continue
        view = bucket[int(g["off"]):int(g["off"]) + int(g["bytes"])]
        if me == a:
            ops.append(dist.P2POp(dist.isend, view, b))
            sent += int(g["bytes"])
        elif me == b:
            ops.append(dist.P2POp(dist.irecv, view, a))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    return sent


def sharded_round(plan, rnd: int, bucket: torch.Tensor, dist, trainer_owner: Sequence[int],
                  rollout_owner: Sequence[int], me: int, stream: int = 0) -> None:
    """One round of the rank-sharded transfer on this process's GPU: pack the slabs of the trainer
    ranks it owns, exchange regions, assemble the parameters of the rollout ranks it owns.  The plan
    must be bound with this process's addresses for the tensors of its own ranks; a payload that is
    replicated on rollout ranks of another process is written through whatever address that tensor
    was bound with (a peer mapping).  Not run on more than one GPU here: one GPU per call."""
    mine_t = [v for v, p in enumerate(trainer_owner) if p == me]
    mine_r = [v for v, p in enumerate(rollout_owner) if p == me]
    plan.pack_ranks(rnd, mine_t, bucket.data_ptr(), stream)
    if dist is not None:
        torch.cuda.current_stream().synchronize()
        exchange_regions(dist, bucket, plan.bucket_regions(rnd), trainer_owner, rollout_owner, me)
    plan.unpack_ranks(rnd, mine_r, bucket.data_ptr(), stream)
