"""Sharding of a batch of ranking requests over several GPUs (one process per GPU).

Users are independent (the user-side module runs once per request, Sec. 3.3 of the paper), so a batch is split by
user with no collective on the data path: every rank holds the model (links, layer weights, embedding table), gets
a contiguous range of users together with their candidate rows, and runs the single-GPU path on it.  This module
holds the host logic only: the balanced partition, the ragged slices each rank takes, the max-over-ranks timing
reduction and the optional gather of logits.  It works with any torch.distributed backend (nccl on GPUs, gloo in
the CPU tests).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


def user_costs(lengths: Sequence[int], cands_per_user: Sequence[int], ell: int, n_layers: int) -> np.ndarray:
    """Relative cost of each user: history tokens stream through every XOR layer (cost linear in N(U), Sec. 3.2) and
    candidates stream once through the scorer (cost linear in M(U)); both per-unit costs scale with the link count."""
    n = np.asarray(lengths, dtype=np.int64)
    c = np.asarray(cands_per_user, dtype=np.int64)
    return (n * int(n_layers) * 2 + c) * int(ell)


def partition_users(costs: Sequence[int], world: int) -> List[Tuple[int, int]]:
    """Contiguous user ranges [lo, hi) per rank, balanced by cumulative cost: rank r ends at the first user whose
    cumulative cost reaches (r + 1) / world of the total.  Every user belongs to exactly one rank; ranks may be empty
    when there are fewer users than ranks."""
    costs = np.asarray(costs, dtype=np.float64)
    B = int(costs.size)
    if world <= 0:
        raise ValueError("world must be positive")
    cum = np.concatenate([[0.0], np.cumsum(costs)])
    total = cum[-1]
    bounds = [0]
    for r in range(1, world):
        if total <= 0:
            cut = (B * r) // world
        else:
            cut = int(np.searchsorted(cum, total * r / world, side="left"))
        bounds.append(min(B, max(bounds[-1], cut)))
    bounds.append(B)
    return [(bounds[r], bounds[r + 1]) for r in range(world)]


def shard_slices(lengths: Sequence[int], cand_counts: Sequence[int], lo: int, hi: int):
    """Token and candidate slices of users [lo, hi) in the batch-wide ragged arrays."""
    n = np.asarray(lengths, dtype=np.int64)
    c = np.asarray(cand_counts, dtype=np.int64)
    t0, t1 = int(n[:lo].sum()), int(n[:hi].sum())
    c0, c1 = int(c[:lo].sum()), int(c[:hi].sum())
    return slice(t0, t1), slice(c0, c1)


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """The slowest rank's value (all_reduce MAX); identity in a single process."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_this_rank: float, seconds_this_rank: float, device: Optional[torch.device] = None) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)


def gather_logits(local: torch.Tensor, counts: Sequence[int]) -> torch.Tensor:
    """Concatenate the ranks' logits in rank order (= user order, since the partition is contiguous).  `counts[r]` is
    the number of logits rank r holds; ranks pad to the largest count for the fixed-size all_gather."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    width = int(max(counts)) if len(counts) else 0
    buf = torch.zeros(width, dtype=local.dtype, device=local.device)
    buf[: local.numel()] = local
    out = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(out, buf)
    return torch.cat([out[r][: int(counts[r])] for r in range(world)])
