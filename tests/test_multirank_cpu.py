"""world_size-2 (and 3) gloo tests of the multi-rank path: range sharding of a
fragment, combination of per-rank records, and max-over-ranks timing.  The
per-rank merge is done by the oracle here (no GPU in this suite); the plumbing
under test is the same code bench.py and a sharded deployment use."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2604_21428_b200 import dist as ddist
from paper_2604_21428_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_shard_range_partitions_exactly():
    for n in (0, 1, 7, 8, 9, 1000, 8191, 8192, 500_000_000):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                lo, hi = ddist.shard_range(n, r, world)
                assert lo == prev and lo <= hi <= n
                assert lo % 8 == 0 or lo == n
                prev = hi
            assert prev == n
    sizes = [ddist.shard_range(1000, r, 3)[1] - ddist.shard_range(1000, r, 3)[0] for r in range(3)]
    assert max(sizes) - min(sizes) <= 8
    with pytest.raises(ValueError):
        ddist.shard_range(10, 2, 2)


def _worker(rank, world, port, n, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M, tokens, mask, K = 5, [100, 0, 300, 400, 500], 0b11101, 3
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", seed=77)       # same on every rank
        lo, hi = ddist.shard_range(n, rank, world)
        t_s, v_s = theta[lo:hi].copy(), v[lo:hi].copy()
        l_s = [a[lo:hi].copy() for a in learners]
        rec = oracle.merge_fragment(t_s, v_s, l_s, tokens, mask, K, 0.7, 0.9)
        rec = ddist.allreduce_record(rec)
        slowest = ddist.max_over_ranks(10.0 + rank)
        # gather the shards on rank 0 and compare with the unsharded merge
        parts = [None] * world
        dist.all_gather_object(parts, (lo, hi, t_s, v_s))
        if rank == 0:
            t_full, v_full = np.empty_like(theta), np.empty_like(v)
            for a, b, ts, vs in parts:
                t_full[a:b], v_full[a:b] = ts, vs
            ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, 0.7, 0.9)
            ok = (np.array_equal(t_full, theta) and np.array_equal(v_full, v)
                  and rec.idx == ref.idx and rec.w_hat == ref.w_hat and rec.status == ref.status
                  and abs(rec.delta_sq - ref.delta_sq) <= 1e-12 * ref.delta_sq
                  and abs(rec.theta_sq - ref.theta_sq) <= 1e-12 * ref.theta_sq
                  and abs(rec.mom_sq - ref.mom_sq) <= 1e-12 * ref.mom_sq
                  and all(abs(a - b) <= 1e-12 * b for a, b in zip(rec.delta_m_sq, ref.delta_m_sq))
                  and slowest == 10.0 + world - 1)
            out.put(bool(ok))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,n", [(2, 10_007), (3, 4_096), (2, 5)])
def test_range_sharded_merge_equals_unsharded(world, n):
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get() is True


def test_whole_job_rate():
    assert ddist.whole_job_rate(500, 4, 2, 1000.0) == 4000.0
    assert ddist.max_over_ranks(3.5) == 3.5          # no process group: identity


class _FakePassCtx:
    """Stands in for the GPU passes of a range-sharded radial-directional merge: each pass writes
    this rank's share of the fields it hands over and checks that the previous hand-over has been
    summed over the ranks before it runs."""

    def __init__(self, rank, world, dd):
        self.rank, self.world, self.dd, self.calls = rank, world, dd, []

    def _table(self, records):
        return records.view(torch.float64).view(-1, self.dd.RECORD_BYTES // 8)

    def merge_fragments_batched_rda_pass(self, fragments, M, learner_dtype, lr, mu, pass_index, *, records,
                                         scratch, merge_kinds=None, flags=0, push_masks=None, stream=None):
        dd, t, r = self.dd, self._table(records), self.rank
        total = sum(range(1, self.world + 1))
        a, b = dd.record_field_columns("delta_m_sq")
        c, _ = dd.record_field_columns("delta_sq")
        if pass_index == dd.RDA_PASS_NORMS:
            t[:, a:a + M] = torch.arange(M, dtype=torch.float64) + (r + 1)
        elif pass_index == dd.RDA_PASS_DIRECTION:
            assert torch.equal(t[0, a:a + M], torch.arange(M, dtype=torch.float64) * self.world + total)
            t[:, c] = 10.0 * (r + 1)
        else:
            assert float(t[0, c]) == 10.0 * total
            assert torch.equal(t[0, a:a + M], torch.arange(M, dtype=torch.float64) * self.world + total)
            for k, name in enumerate(("delta_sq", "theta_sq", "mom_sq")):
                t[:, dd.record_field_columns(name)[0]] = (k + 1.0) * (r + 1)
        self.calls.append(pass_index)


def _rda_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2604_21428_b200 import ddmerge as dd
        P, M = 3, 4
        records = torch.zeros(P * dd.RECORD_BYTES, dtype=torch.uint8)
        ctx = _FakePassCtx(rank, world, dd)
        ddist.rda_merge_range_sharded(ctx, [None] * P, M, dd.BF16, 0.7, 0.9, records=records,
                                      scratch=torch.zeros(8))
        t = records.view(torch.float64).view(P, dd.RECORD_BYTES // 8)
        total = sum(range(1, world + 1))
        ok = ctx.calls == [dd.RDA_PASS_NORMS, dd.RDA_PASS_DIRECTION, dd.RDA_PASS_APPLY]
        for k, name in enumerate(("delta_sq", "theta_sq", "mom_sq")):
            ok = ok and bool(torch.all(t[:, dd.record_field_columns(name)[0]] == (k + 1.0) * total))
        a, _ = dd.record_field_columns("delta_m_sq")
        # the norms were summed once, after the first pass, and not again at the end
        ok = ok and torch.equal(t[1, a:a + M], torch.arange(M, dtype=torch.float64) * world + total)
        out[rank] = bool(ok)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_range_sharded_rda_hands_over_between_passes(world):
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rda_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert all(out[r] for r in range(world)) and len(out) == world


class _OraclePassCtx:
    """The three passes of a range-sharded radial-directional merge done by the ORACLE on this rank's
    element range, behind the interface of the library's per-pass call: each pass reads the hand-over
    fields that the previous all-reduce left in the records buffer and writes its own share."""

    def __init__(self, dd, shards):
        self.dd, self.shards = dd, shards          # shards[p] = (theta, v, learners) of this rank's range

    def _table(self, records):
        return records.view(torch.float64).view(-1, self.dd.RECORD_BYTES // 8)

    def merge_fragments_batched_rda_pass(self, fragments, M, learner_dtype, lr, mu, pass_index, *, records,
                                         scratch, merge_kinds=None, flags=0, push_masks=None, stream=None):
        dd, t = self.dd, self._table(records)
        a, _ = dd.record_field_columns("delta_m_sq")
        c, _ = dd.record_field_columns("delta_sq")
        for p, f in enumerate(fragments):
            theta, v, learners = self.shards[p]
            st, idx = oracle.participants(f["quorum_mask"], f["tokens"], f["K"])
            s = len(idx)
            norms = [float(x) for x in t[p, a:a + s]]
            rec, dsq = oracle.merge_fragment_rda_stage(pass_index, theta, v, learners, f["tokens"],
                                                       f["quorum_mask"], f["K"], lr, mu,
                                                       norms_sq=norms if pass_index > 0 else None,
                                                       dir_sq=float(t[p, c]) if pass_index == 2 else 0.0)
            if pass_index == 0:
                t[p, a:a + s] = torch.tensor(rec.delta_m_sq, dtype=torch.float64)
            elif pass_index == 1:
                t[p, c] = dsq
            else:
                for name in ("delta_sq", "theta_sq", "mom_sq"):
                    t[p, dd.record_field_columns(name)[0]] = getattr(rec, name)


def _rda_oracle_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2604_21428_b200 import ddmerge as dd
        M, K = 5, 2
        sizes = [10_007, 4_099]
        tokens = [[100, 0, 300, 400, 500], [7, 9, 11, 0, 13]]
        masks = [0b11101, 0b10111]
        whole, shards, frags, ranges = [], [], [], []
        for p, n in enumerate(sizes):
            theta, v, learners = synth.fragment_cpu(n, M, "bf16", seed=900 + p)     # same on every rank
            v[:] = np.random.default_rng(p).normal(0, 1e-4, n).astype(np.float32)
            whole.append((theta, v, learners))
            lo, hi = ddist.shard_range(n, rank, world)
            ranges.append((lo, hi))
            shards.append((theta[lo:hi].copy(), v[lo:hi].copy(), [a[lo:hi].copy() for a in learners]))
            frags.append(dict(tokens=tokens[p], quorum_mask=masks[p], K=K, n=hi - lo))
        records = torch.zeros(len(sizes) * dd.RECORD_BYTES, dtype=torch.uint8)
        ddist.rda_merge_range_sharded(_OraclePassCtx(dd, shards), frags, M, dd.BF16, 0.7, 0.9,
                                      records=records, scratch=torch.zeros(8))
        parts = [None] * world
        dist.all_gather_object(parts, [(ranges[p], shards[p][0], shards[p][1]) for p in range(len(sizes))])
        ok = True
        t = records.view(torch.float64).view(len(sizes), dd.RECORD_BYTES // 8)
        for p, n in enumerate(sizes):
            theta, v, learners = whole[p]
            ref = oracle.merge_fragment(theta, v, learners, tokens[p], masks[p], K, 0.7, 0.9,
                                        merge=oracle.MERGE_RDA)
            t_full, v_full = np.empty(n, np.float32), np.empty(n, np.float32)
            for per_rank in parts:
                (lo, hi), ts, vs = per_rank[p]
                t_full[lo:hi], v_full[lo:hi] = ts, vs
            # the shards' sums are taken in another order than the whole fragment's: a few ulps of
            # the norms, hence of Delta, hence at most an ulp or two of the float32 state
            ok = ok and float(np.max(np.abs(t_full - theta))) <= 2e-9 and float(np.max(np.abs(v_full - v))) <= 1e-9
            for name in ("delta_sq", "theta_sq", "mom_sq"):
                got = float(t[p, dd.record_field_columns(name)[0]])
                ok = ok and abs(got - getattr(ref, name)) <= 1e-10 * getattr(ref, name)
            a, _ = dd.record_field_columns("delta_m_sq")
            ok = ok and all(abs(float(t[p, a + j]) - x) <= 1e-12 * x for j, x in enumerate(ref.delta_m_sq))
        out[rank] = bool(ok)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_range_sharded_rda_with_oracle_shards_equals_whole_fragment(world):
    """dist.rda_merge_range_sharded on gloo ranks, every rank's passes computed by the oracle on
    its own element range: after the two all-reduces the gathered fragment equals the oracle's
    radial-directional merge of the whole fragment, and every rank holds whole-fragment norms."""
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_rda_oracle_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert all(out[r] for r in range(world)) and len(out) == world
