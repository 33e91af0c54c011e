"""Multi-GPU plumbing for the merge: how a fragment is split across ranks and how
per-rank results are combined.  The merge is element-wise, so the data path needs
no collective: a rank owns a contiguous element range of the global fragment, of
the momentum and of every learner copy.  Only scalars cross ranks -- the squared
norms of the diagnostics (one small all-reduce) and the timing of a benchmark.
Works on any ``torch.distributed`` backend (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

import dataclasses


def shard_range(n: int, rank: int, world: int, align: int = 8):
    """Contiguous element range [lo, hi) of rank ``rank``; interior boundaries are
    multiples of ``align`` elements so every shard starts 16-byte aligned."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = (n + align - 1) // align
    base, extra = divmod(units, world)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(lo_u * align, n), min(hi_u * align, n)


def max_over_ranks(value: float, device=None, group=None) -> float:
    """MAX all-reduce of one float (benchmark time of the slowest rank)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def allreduce_record(rec, device=None, group=None):
    """Combines the records of a range-sharded merge: participation and weights are
    identical on every rank (they depend only on mask and counters); squared
    norms are sums over the ranks' element ranges."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return rec
    s = len(rec.delta_m_sq)
    vals = [rec.delta_sq, rec.theta_sq, rec.mom_sq] + list(rec.delta_m_sq)
    t = torch.tensor(vals, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    status = torch.tensor([rec.status], dtype=torch.int64, device=device)
    dist.all_reduce(status, op=dist.ReduceOp.MAX, group=group)
    out = t.tolist()
    return dataclasses.replace(rec, status=int(status.item()), delta_sq=out[0], theta_sq=out[1],
                               mom_sq=out[2], delta_m_sq=out[3:3 + s])


def whole_job_rate(units_per_rank_step: int, steps: int, world: int, max_ms: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return world * units_per_rank_step * steps / (max_ms * 1e-3)
