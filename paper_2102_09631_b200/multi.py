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


def allgather_factors(P_local: torch.Tensor, Q_local: torch.Tensor, n_sites: int):
    """The one exchange step of rank-dAD when the S sites are sharded over ranks (`shard_units`): every rank
    contributes the factors of its own sites and receives the stacks of all of them, in site order -- the
    aggregator's vertcat followed by the broadcast, as one all-gather into each rank's own memory.

    P_local: S_local x r x h_in, Q_local: S_local x r x h_out (this rank's sites, in order; S_local may differ
    by one between ranks).  Returns (Pcat, Qcat) of n_sites*r rows each.  Works on CPU tensors with gloo and on
    CUDA tensors with nccl; a single process returns its own factors reshaped."""
    r, h_in, h_out = P_local.shape[1], P_local.shape[2], Q_local.shape[2]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        assert P_local.shape[0] == n_sites
        return P_local.reshape(n_sites * r, h_in), Q_local.reshape(n_sites * r, h_out)
    world, rank = dist.get_world_size(), dist.get_rank()
    counts = [len(shard_units(n_sites, k, world)) for k in range(world)]
    assert P_local.shape[0] == counts[rank] == Q_local.shape[0]
    cap = max(counts)
    # one buffer per rank holding P then Q, padded to the largest shard so that all contributions have one size
    mine = torch.zeros(cap * r * (h_in + h_out), dtype=P_local.dtype, device=P_local.device)
    nP, nQ = counts[rank] * r * h_in, counts[rank] * r * h_out
    mine[:nP] = P_local.reshape(-1)
    mine[cap * r * h_in:cap * r * h_in + nQ] = Q_local.reshape(-1)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    Ps = [parts[k][:counts[k] * r * h_in].reshape(counts[k] * r, h_in) for k in range(world)]
    Qs = [parts[k][cap * r * h_in:cap * r * h_in + counts[k] * r * h_out].reshape(counts[k] * r, h_out)
          for k in range(world)]
    return torch.cat(Ps), torch.cat(Qs)


class SiteShardedLayer:
    """One linear layer whose S sites are dealt over the ranks (`shard_units`): rank k compresses its own sites,
    one all-gather of the fp32 factors lands the stacks of ALL sites in every rank's own memory (Algorithm 1's
    vertcat at the aggregator and its broadcast back, as a single exchange), and every rank reconstructs the same
    gradient locally.  The arithmetic is supplied by the caller -- the library's calls on CUDA tensors over nccl, or
    any stand-in on CPU tensors over gloo -- so that this exchange logic is the same code in both settings:

        compress(site_indices) -> (P_local, Q_local)   S_local x r x h_in / h_out, this rank's sites in order
        reconstruct(Pcat, Qcat) -> gradient             from the (S*r)-row stacks

    `sent_bytes` is what this rank contributes to the exchange for one layer: r*(h_in+h_out)*4 per own site, the
    rank-dAD transmission count of those sites."""

    def __init__(self, n_sites: int, r: int, h_in: int, h_out: int):
        rank, world = (dist.get_rank(), dist.get_world_size()) if (dist.is_available() and dist.is_initialized()) else (0, 1)
        self.n_sites, self.r, self.h_in, self.h_out = n_sites, r, h_in, h_out
        self.rank, self.world = rank, world
        self.sites = shard_units(n_sites, rank, world)
        self.sent_bytes = len(self.sites) * r * (h_in + h_out) * 4

    def step(self, compress, reconstruct, on_exchange=None):
        P_local, Q_local = compress(self.sites)
        if on_exchange is not None:
            on_exchange(True)
        Pcat, Qcat = allgather_factors(P_local, Q_local, self.n_sites)
        if on_exchange is not None:
            on_exchange(False)
        return reconstruct(Pcat, Qcat)
