"""Host-side helpers for running the layer path on several GPUs of one node.

The path shards by independent units (sites, layers): every rank processes its own batch of the
same shape and nothing crosses GPUs on the data path.  What the ranks share is only the
measurement protocol: a barrier on both sides of the timed region and the maximum of the
per-rank device times.  These helpers work with any torch.distributed backend (nccl on GPUs,
gloo in the CPU tests).
"""
from __future__ import annotations

import os
from typing import List, Sequence

import torch
import torch.distributed as dist


def env_rank_world() -> tuple:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None) -> None:
    """Join the process group described by MASTER_ADDR/MASTER_PORT/RANK/WORLD_SIZE (no-op for one rank)."""
    rank, _, world = env_rank_world()
    if world > 1 and not dist.is_initialized():
        kwargs = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kwargs)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what the whole job took."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, seconds: float) -> float:
    """Units all ranks processed per second (weak scaling: every rank does `units_per_rank`)."""
    return units_per_rank * world / seconds


def shard_units(n_units: int, rank: int, world: int) -> List[int]:
    """Strong-scaling split of n_units independent units (sites or layers): contiguous, sizes differ by <= 1."""
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def gather_counts(local: Sequence[int]) -> List[List[int]]:
    """All ranks' integer lists (e.g. per-site byte counts) on every rank, in rank order."""
    if not (dist.is_available() and dist.is_initialized()):
        return [list(local)]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, list(local))
    return out
