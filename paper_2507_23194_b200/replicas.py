"""Rank bookkeeping for running the verifier on several GPUs of one node.

The path does not shard below one GPU (`one GPU only`): candidates are independent, so N GPUs run N
replicas, or split the candidate list of one batch among themselves, with no collective on the data
path. What the ranks do share is bookkeeping, and that is all this module holds (no arithmetic of the
verifier): which candidates a rank owns, the slowest rank's time, and the gathered 64-byte records.
It works with any `torch.distributed` backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard_candidates(n_cands: int, world: int, rank: int) -> List[int]:
    """Indices of the candidates rank `rank` verifies when one batch is split over `world` ranks:
    contiguous, sizes differing by at most one, every index owned exactly once."""
    if world < 1 or not (0 <= rank < world) or n_cands < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_cands, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def shard_plan(n_cands: int, world: int, rank: int):
    """(records per rank in rank order, this rank's candidate indices) for one batch split over `world` ranks."""
    return [len(shard_candidates(n_cands, world, r)) for r in range(world)], shard_candidates(n_cands, world, rank)


def verify_sharded(ref, cands, verify_local, world: int, rank: int) -> torch.Tensor:
    """One batch, candidates split among the ranks: this rank verifies its own share with `verify_local(ref,
    cands_of_this_rank) -> uint8 [n, 64]` (the CUDA library's dense call on a GPU; any stand-in with the same
    contract on CPU ranks) and every rank receives the records of the whole batch in candidate order."""
    counts, mine = shard_plan(len(cands), world, rank)
    local = verify_local(ref, [cands[j] for j in mine])
    if local.shape[0] != len(mine):
        raise ValueError("verify_local returned a different number of records than candidates it was given")
    return gather_records(local, counts)


def max_over_ranks(ms: float, device="cpu") -> float:
    """The slowest rank's time (what a multi-GPU number must be quoted on)."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_records(local: torch.Tensor, counts: Sequence[int]) -> torch.Tensor:
    """Concatenate the ranks' record blocks (uint8 [n_r, 64]) in rank order on every rank.
    `counts[r]` is rank r's number of records."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    width = max(counts) if counts else 0
    padded = torch.zeros((width, 64), dtype=torch.uint8, device=local.device)
    padded[: local.shape[0]] = local
    out = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(out, padded)
    return torch.cat([o[: counts[r]] for r, o in enumerate(out)], dim=0)


def aggregate_throughput(bytes_per_rank: int, ms: float) -> float:
    """Whole-job GB/s when every rank processed `bytes_per_rank` in `ms` (max over ranks)."""
    world = dist.get_world_size() if dist.is_initialized() else 1
    return world * bytes_per_rank / (ms * 1e-3) / 1e9
