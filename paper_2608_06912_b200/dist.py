"""Multi-GPU plumbing for the benchmark and for row-sharded batches.

Rows are independent problems, so a batch shards by rows with no collective
(each rank owns a contiguous slice and runs the same kernels on it).  ONE row
can also be spread over several GPUs: forward_sharded / backward_sharded drive
the per-shard steps (a shard object per contiguous piece of the row) and merge
what they leave behind with three small exchanges - a sum of the sample's key
buffers, a sum of tails / counts / bucket tables plus a concatenation of the
bands, and a sum of the four VJP sums.  The exchanges are torch.distributed
collectives between processes (NCCL on GPUs, gloo in the CPU tests) and plain
tensor sums between the shards one process holds; the same code serves both,
so several shards in ONE process on one GPU exercise the whole path.
"""
from __future__ import annotations

import os
from typing import Callable, List, Optional, Sequence, Tuple

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


# ------------------------------------------------------------ one row over several GPUs ----
def _group_active(group) -> bool:
    return dist.is_available() and dist.is_initialized() and (group is not None or dist.get_world_size() > 1)


def _sum_over_shards(shards: Sequence, name: str, group=None) -> None:
    """Every shard's tensor `name` <- the sum of that tensor over all shards of all ranks (rank order, then shard order)."""
    first = getattr(shards[0], name)
    total = first.clone()
    for s in shards[1:]:
        total += getattr(s, name)
    if _group_active(group):
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    for s in shards:
        getattr(s, name).copy_(total)


def _merge_bands(shards: Sequence, counts_local: List[int], group=None) -> int:
    """Every shard's band buffer <- the bands of all shards of all ranks, one after the other; returns the total count
    (the buffers are left alone when the total exceeds their capacity: the solve then reports the overflow)."""
    cap = shards[0].band_capacity
    pieces = [s.band_keys[: min(c, cap)] for s, c in zip(shards, counts_local)]
    local = torch.cat(pieces) if len(pieces) > 1 else pieces[0].clone()
    total = sum(counts_local)
    if _group_active(group):
        world = dist.get_world_size(group)
        mine = torch.tensor([local.numel(), total], dtype=torch.int64, device=local.device)
        every = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(every, mine, group=group)
        sizes = [int(t[0]) for t in every]   # host read: the concatenation needs the sizes
        total = sum(int(t[1]) for t in every)
        longest = max(sizes + [1])
        padded = torch.zeros(longest, dtype=local.dtype, device=local.device)
        padded[: local.numel()] = local
        gathered = [torch.empty_like(padded) for _ in range(world)]
        dist.all_gather(gathered, padded, group=group)
        local = torch.cat([g[:sz] for g, sz in zip(gathered, sizes)])
    if total <= cap:
        for s in shards:
            s.band_keys[: local.numel()].copy_(local)
    return total


def forward_sharded(shards: Sequence, k: float, alpha: float, group=None, gather_row: Optional[Callable] = None) -> bool:
    """Forward of ONE row whose contiguous pieces are `shards` (this process's, in row order; other ranks of `group`
    hold the rest).  Leaves the mask of every shard in shard.p and the row's threshold in shard.b.  Returns True when
    the bracket held; on a failed certificate (about once in 10^6 calls at z = 5.16) the row is gathered through
    gather_row() and every shard falls back to the ordinary forward of the whole row: returns False."""
    for s in shards:
        s.sample(alpha)
    _sum_over_shards(shards, "sample_keys", group)
    for s in shards:
        s.stream_pass(k, alpha)
    counts = [int(s.band_count.item()) for s in shards]       # host read (also orders the stream passes before the merge)
    for name in ("tails", "n_R", "bucket_counts", "bucket_sums"):
        _sum_over_shards(shards, name, group)
    total = _merge_bands(shards, counts, group)
    for s in shards:
        s.band_count.fill_(total)
        s.solve(k, alpha)
    held = not bool(torch.isnan(shards[0].b).item())           # identical on every rank: same inputs, same arithmetic
    if held:
        for s in shards:
            s.mask(alpha)
        return True
    if gather_row is None:
        raise RuntimeError("the bracket's certificate failed and no gather_row() was given for the whole-row fallback")
    r_full = gather_row()
    for s in shards:
        s.whole_row_forward(r_full, k, alpha)
    return False


def backward_sharded(shards: Sequence, v_shards: Sequence, alpha: float, group=None) -> None:
    """Backward of the row of forward_sharded: v_shards are the pieces of the upstream gradient; leaves shard.grad,
    shard.grad_k and shard.grad_alpha (the scalars are those of the whole row, the same on every shard)."""
    for s, v in zip(shards, v_shards):
        s.vjp_partial(v, alpha)
    _sum_over_shards(shards, "vjp_sums", group)
    for s, v in zip(shards, v_shards):
        s.vjp_apply(v, alpha)


def gather_row_over(shards: Sequence, group=None) -> Callable:
    """gather_row() for forward_sharded: concatenates the local shards and, between processes, all-gathers them
    (shards of equal length per rank are assumed for the collective)."""
    def gather():
        local = torch.cat([s.r.view(-1) for s in shards])
        if not _group_active(group):
            return local
        world = dist.get_world_size(group)
        parts = [torch.empty_like(local) for _ in range(world)]
        dist.all_gather(parts, local, group=group)
        return torch.cat(parts)
    return gather


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
