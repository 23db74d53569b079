"""Multi-GPU plumbing for the benchmark and for row-sharded batches.

The solver has no data-path collective: rows are independent problems, so a
batch shards by rows (each rank owns a contiguous slice and runs the same
kernels on it), and a single huge row runs as independent replicas.  The only
cross-rank traffic is the timing protocol (barrier, max over ranks).
"""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when not launched by torchrun."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float, device: torch.device) -> float:
    """Largest value of x on any rank (the step time of a multi-GPU run is the slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device: torch.device) -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def row_shard(rows: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous [lo, hi) slice of `rows` owned by `rank`: sizes differ by at most one, nothing is dropped."""
    base, extra = divmod(rows, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo, hi


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
