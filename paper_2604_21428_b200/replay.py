"""Syncer loop (Algorithm 2) driven by a recorded or synthetic event tape.

A tape fixes, for every syncer step, when each learner's report arrived and the
per-(learner, fragment) token / step counters it carried -- exactly what the
paper's deterministic replay records ("participant subsets and token
weightings").  ``Syncer.step`` turns one tape entry into library calls: quorum
selection with the grace window, ONE batched merge launch over the fragments that
are due, and the push of the updated fragments to the learners that are alive --
inside the merge launch when the learners simply take the new fragment (alpha = 0),
as a broadcast launch per fragment otherwise.  All arithmetic
happens in libddmerge; this module only sequences calls.
"""
from __future__ import annotations

from dataclasses import dataclass, field

from . import ddmerge as dd


@dataclass
class TapeEntry:
    arrival_s: list                 # M arrival times of the reports (inf = no report)
    tokens: list                    # P x M counters since the learner last received fragment p
    steps: list | None = None       # P x M, optional


@dataclass
class StepResult:
    due: list = field(default_factory=list)
    mask: int = 0
    n_admitted: int = 0
    records: list = field(default_factory=list)


class Syncer:
    """Holds the global fragments and the outer momentum on one GPU."""

    def __init__(self, ctx: "dd.Context", global_fragments, momentum_fragments, *, H: int,
                 offsets, K: int, outer_lr: float, outer_mu: float, learner_dtype: int,
                 merge_kinds=None, alpha: float = 0.0, flags: int = 0, fused_push: bool = True):
        self.ctx = ctx
        self.theta = list(global_fragments)
        self.mom = list(momentum_fragments)
        self.P = len(self.theta)
        self.H, self.offsets, self.K = int(H), list(offsets), int(K)
        self.lr, self.mu = float(outer_lr), float(outer_mu)
        self.dtype = learner_dtype
        self.kinds = list(merge_kinds) if merge_kinds is not None else [dd.MERGE_AVG] * self.P
        self.alpha = float(alpha)
        self.flags = int(flags)
        self.fused_push = bool(fused_push)
        self._records = dd.new_records(self.P, device=self.theta[0].device)

    def due(self, t: int):
        """Fragments synchronised at step t: those with t mod H equal to their offset."""
        return [p for p in range(self.P) if t % self.H == self.offsets[p]]

    def step(self, t: int, entry: TapeEntry, learner_fragments, grace_s: float = 0.0,
             stream=None, read_back: bool = True) -> StepResult:
        """``learner_fragments[m][p]`` is learner m's device copy of fragment p (or None).

        ``read_back=False`` keeps the step asynchronous: the records stay on the device and
        the decision to broadcast is taken from what the host already knows (enough
        admitted learners with a positive token count), which is the kernel's own test."""
        res = StepResult(due=self.due(t))
        if not res.due:
            return res
        M = len(entry.arrival_s)
        res.mask, res.n_admitted = dd.select_quorum(entry.arrival_s, self.K, grace_s)
        frags = []
        for p in res.due:
            frags.append(dict(global_=self.theta[p], momentum=self.mom[p],
                              learners=[learner_fragments[m][p] for m in range(M)],
                              tokens=entry.tokens[p],
                              steps=None if entry.steps is None else entry.steps[p],
                              quorum_mask=res.mask, K=self.K, n=int(self.theta[p].numel())))
        recs = self._records[: len(frags) * dd.RECORD_BYTES]
        kinds = [self.kinds[p] for p in res.due]
        # every learner that is alive receives the new fragment (and resets its counters)
        alive = sum(1 << m for m in range(M) if entry.arrival_s[m] != float("inf"))
        has_rda = any(k == dd.MERGE_RDA for k in kinds)
        fused = self.fused_push and self.alpha == 0.0 and alive != 0
        if has_rda:
            self.ctx.merge_fragments_batched_rda(frags, M, self.dtype, self.lr, self.mu,
                                                 merge_kinds=kinds, flags=self.flags, records=recs,
                                                 stream=stream,
                                                 push_masks=[alive] * len(frags) if fused else None)
        elif fused:
            # merge and push in one launch; a fragment whose quorum is not met pushes nothing
            self.ctx.merge_fragments_batched_push(frags, [alive] * len(frags), M, self.dtype, self.lr,
                                                  self.mu, flags=self.flags, records=recs, stream=stream)
        else:
            self.ctx.merge_fragments_batched(frags, M, self.dtype, self.lr, self.mu,
                                             flags=self.flags, records=recs, stream=stream)
        if read_back:
            res.records = dd.read_records(recs, len(frags))
            merged = [rec.status == dd.STATUS_OK for rec in res.records]
        elif not fused:
            need = max(self.K, 1)
            merged = [sum(1 for m in range(M) if (res.mask >> m) & 1 and entry.tokens[p][m] > 0) >= need
                      for p in res.due]
        if not fused:
            for p, ok in zip(res.due, merged):
                if ok and alive:
                    self.ctx.broadcast_fragment(self.theta[p],
                                                [learner_fragments[m][p] for m in range(M)], alive,
                                                self.alpha, n=int(self.theta[p].numel()),
                                                learner_dtype=self.dtype, stream=stream)
        return res
