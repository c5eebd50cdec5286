"""Multi-process plumbing for the benchmark: the hot path shards by independent graph
batches (one process per GPU, no data-path collective), so the only communication is the
barrier around the timed region and the max-over-ranks / sum-over-ranks of the results."""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment (1 process: 0, 0, 1)."""
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init_process_group(backend: str) -> Optional[dist.ProcessGroup]:
    rank, _, world = env_world()
    if world == 1:
        return None
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return dist.group.WORLD


def barrier(device: torch.device) -> None:
    if dist.is_initialized():
        if device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def aggregate(ms_local: float, units_local: float, device: torch.device) -> Tuple[float, float]:
    """Whole-job figures: (max over ranks of the elapsed milliseconds, sum over ranks of the
    units processed).  With one process it is the identity."""
    if not dist.is_initialized():
        return ms_local, units_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def shard_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own batch (weak scaling over independent graph batches)."""
    return base_seed + 1009 * rank
