"""Host-side helpers for running the path on several GPUs of one node.

Every (batch, head) pair is an independent unit of the forward, the decode and of dQ / dK / dV, so the
path shards by units with no collective on the data path; the only cross-rank traffic is the barrier
and the max-reduction of the measured step time (and, if the heads of one batch element were split,
a sum of the small gate gradients dG [B, T, 3] and dW_r [D, 3]).  Nothing here touches CUDA: the same
code runs under the `gloo` backend on CPU ranks, which is how it is tested.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def shard_units(total: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced split of `total` units over `world` ranks: (first unit, number of units) of `rank`.
    The first `total % world` ranks get one unit more; every unit belongs to exactly one rank."""
    if world <= 0 or not 0 <= rank < world or total < 0:
        raise ValueError("invalid shard request")
    base, extra = divmod(total, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def shard_batch_heads(B: int, H: int, world: int, rank: int) -> List[Tuple[int, int, int]]:
    """The (batch, first head, number of heads) slices that make up `rank`'s share of the B*H units."""
    start, count = shard_units(B * H, world, rank)
    out, u, end = [], start, start + count
    while u < end:
        b, h = divmod(u, H)
        n = min(H - h, end - u)
        out.append((b, h, n))
        u += n
    return out


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Step time of the job = the slowest rank's (all-reduce MAX); the identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(t: torch.Tensor, dist=None) -> torch.Tensor:
    """In-place sum of a small gradient tensor (dG, dW_r) over ranks; the identity without a process group."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def job_throughput(units_per_rank_work: float, world: int, step_ms_max: float) -> float:
    """Whole-job rate under weak scaling: every rank does `units_per_rank_work` per step, the step takes the max."""
    return world * units_per_rank_work / (step_ms_max * 1e-3)
