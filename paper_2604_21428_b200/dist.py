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


# Fields of the device-side records that the passes of a range-sharded radial-directional
# merge hand to one another, and must therefore be summed over the shards before the next pass.
RDA_HANDOVER_FIELDS = {0: ("delta_m_sq",), 1: ("delta_sq",), 2: ("delta_sq", "theta_sq", "mom_sq")}


def sum_record_fields(records, fields, record_bytes: int, columns, reduce_sum) -> None:
    """Sums ``fields`` of a records buffer (uint8 tensor of whole records) over the shards, in
    place.  ``columns(name)`` gives a field's float64 column range, ``reduce_sum(tensor)`` does
    the cross-shard sum in place (an all-reduce; a test may pass its own)."""
    import torch

    table = records.view(torch.float64).view(-1, record_bytes // 8)
    for name in fields:
        a, b = columns(name)
        part = table[:, a:b].contiguous()
        reduce_sum(part)
        table[:, a:b] = part


def rda_merge_range_sharded(ctx, fragments, M: int, learner_dtype: int, outer_lr: float,
                            outer_mu: float, *, records, scratch, merge_kinds=None, flags: int = 0,
                            push_masks=None, stream=None, group=None) -> None:
    """The radial-directional merge of fragments that are sharded by element range: every rank
    calls this with ITS ranges (``fragments`` as for ``merge_fragments_batched_rda``); the three
    passes run one by one and the two whole-fragment quantities the method needs -- the
    participants' norms, then the mean direction's length -- are all-reduced in between
    (a few doubles per fragment, on the device).  Afterwards ``records`` holds whole-fragment
    diagnostics on every rank."""
    import torch.distributed as dist

    from . import ddmerge as dd

    def reduce_sum(t):
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)

    for p in (dd.RDA_PASS_NORMS, dd.RDA_PASS_DIRECTION, dd.RDA_PASS_APPLY):
        ctx.merge_fragments_batched_rda_pass(fragments, M, learner_dtype, outer_lr, outer_mu, p,
                                             records=records, scratch=scratch, merge_kinds=merge_kinds,
                                             flags=flags, push_masks=push_masks, stream=stream)
        sum_record_fields(records, RDA_HANDOVER_FIELDS[p], dd.RECORD_BYTES, dd.record_field_columns,
                          reduce_sum)


def whole_job_rate(units_per_rank_step: int, steps: int, world: int, max_ms: float) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return world * units_per_rank_step * steps / (max_ms * 1e-3)
