"""Radial-directional averaging on the GPU against the oracle's statement of it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import (TOL_BF16, TOL_NORM, TOL_STATE, bf16_bits_to_f32, floor_rel_err,
                         to_torch_learner)

pytestmark = pytest.mark.gpu
ETA, MU = synth.OUTER_LR, synth.OUTER_MU


@pytest.fixture(scope="module")
def dd():
    from paper_2604_21428_b200 import ddmerge
    return ddmerge


@pytest.fixture(scope="module")
def ctx(dd):
    c = dd.Context(0)
    yield c
    c.close()


def _check_record(got, ref):
    assert (got.status, got.n_part, got.idx) == (ref.status, ref.n_part, ref.idx)
    if ref.status != 0:
        return
    assert got.w_hat == [float(np.float32(w)) for w in ref.w_hat]
    for name in ("delta_sq", "theta_sq", "mom_sq"):
        a, b = getattr(got, name), getattr(ref, name)
        assert abs(a - b) <= TOL_NORM * abs(b) + 1e-300, (name, a, b)
    for a, b in zip(got.delta_m_sq, ref.delta_m_sq):
        assert abs(a - b) <= TOL_NORM * abs(b) + 1e-300


def _case(dd, ctx, n, M, dtype, tokens, mask, K, *, seed, steps=None, merges=2, own_scratch=False,
          heavy=False, zero_learner=None, three_pass=False):
    theta, v, learners = synth.fragment_cpu(n, M, dtype, seed)
    if zero_learner is not None:                    # this participant's outer gradient is exactly 0
        if dtype == "bf16":
            theta = oracle.bf16_to_f32(oracle.bf16_rne(theta))
            learners[zero_learner] = oracle.bf16_rne(theta)
        else:
            learners[zero_learner] = theta.copy()
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    out_dev = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    rec_buf = dd.new_records(1)
    scratch = torch.empty((n + 7) // 8 * 8, dtype=torch.float32, device="cuda") if own_scratch else None
    flags = dd.DIAG_STATE | (dd.HEAVY_BALL if heavy else 0) | (dd.RDA_THREE_PASS if three_pass else 0)
    for k in range(merges):
        o_out = np.zeros(n, dtype=np.uint16)
        ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, ETA, MU, steps=steps,
                                    nesterov=not heavy, merge=oracle.MERGE_RDA, out_bf16=o_out)
        ctx.merge_fragment_rda(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU, n=n,
                               learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32, steps=steps,
                               flags=flags, out_bf16=out_dev, record=rec_buf, scratch=scratch)
        torch.cuda.synchronize()
        got = dd.read_records(rec_buf)[0]
        _check_record(got, ref)
        e_t = floor_rel_err(t_dev.cpu().numpy(), theta)
        e_v = floor_rel_err(v_dev.cpu().numpy(), v)
        assert e_t <= TOL_STATE and e_v <= TOL_STATE, (k, e_t, e_v)
        if ref.status == 0:
            assert floor_rel_err(bf16_bits_to_f32(out_dev), oracle.bf16_to_f32(o_out)) <= TOL_BF16
        if n:
            t_dev.copy_(torch.from_numpy(theta))
            v_dev.copy_(torch.from_numpy(v))
    return got


@pytest.mark.parametrize("n", [5, 8, 1023, 8192 * 2 + 3, 200_001])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_rda_sizes(dd, ctx, n, dtype):
    _case(dd, ctx, n, 5, dtype, [100, 200, 0, 400, 500], 0b11101, 2, seed=n % 89)


def test_rda_several_tiles_per_cta(dd, ctx):
    # every pass walks more than one tile per CTA; all elements against the oracle
    _case(dd, ctx, 2 * 296 * 8192 + 8192 + 3, 3, "bf16", [700, 0, 900], 0b111, 2, seed=31, merges=1)


def test_rda_workload_shapes(dd, ctx):
    w = synth.workload("dense150m")
    rec = _case(dd, ctx, 150_003, w.M, "bf16", w.tokens[1].tolist(), w.masks[1], w.K, seed=3,
                own_scratch=True)
    assert rec.n_part == 6
    w = synth.workload("scale500m")
    rec = _case(dd, ctx, 90_000, w.M, "bf16", w.tokens[0].tolist(), w.masks[0], w.K, seed=4, merges=1)
    assert rec.n_part == 24


def test_rda_steps_heavy_ball_and_zero_gradient_participant(dd, ctx):
    _case(dd, ctx, 30_000, 4, "f32", [4000, 9000, 100, 2500], 0b1111, 4, seed=5, steps=[4, 3, 1, 5],
          heavy=True)
    _case(dd, ctx, 30_000, 4, "f32", [5, 5, 5, 5], 0b1111, 1, seed=6, zero_learner=2, merges=1)
    _case(dd, ctx, 30_000, 4, "bf16", [5, 5, 5, 5], 0b1111, 1, seed=6, zero_learner=0, merges=1)


def test_rda_quorum_not_met_touches_nothing(dd, ctx):
    rec = _case(dd, ctx, 10_000, 4, "bf16", [1, 2, 3, 4], 0b0011, 3, seed=7, merges=1)
    assert rec.status == dd.STATUS_QUORUM_NOT_MET


def test_rda_keeps_norm_where_average_shrinks(dd, ctx):
    # near-orthogonal outer gradients of equal norm R: ||RDA|| ~ R, ||Avg|| ~ R / sqrt(M)
    n, M = 1 << 18, 8
    theta, v, learners = synth.fragment_cpu(n, M, "f32", 9)
    t1, v1 = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    t2, v2 = t1.clone(), v1.clone()
    L = [torch.from_numpy(a).cuda() for a in learners]
    r1, r2 = dd.new_records(1), dd.new_records(1)
    ctx.merge_fragment_rda(t1, v1, L, [7] * M, (1 << M) - 1, M, ETA, MU, record=r1)
    ctx.merge_fragment(t2, v2, L, [7] * M, (1 << M) - 1, M, ETA, MU, record=r2,
                       flags=dd.DIAG_PER_LEARNER)
    torch.cuda.synchronize()
    rda, avg = dd.read_records(r1)[0], dd.read_records(r2)[0]
    R = np.sqrt(np.mean(avg.delta_m_sq))
    assert abs(np.sqrt(rda.delta_sq) / R - 1.0) < 0.01
    assert abs(np.sqrt(avg.delta_sq) / (R / np.sqrt(M)) - 1.0) < 0.02


def test_batched_mixed_avg_and_rda(dd, ctx):
    # the paper's policy: direct average on the embedding fragment, RDA elsewhere
    rng = np.random.default_rng(11)
    sizes = [40_003, 8192 * 3, 17, 120_000]
    kinds = [dd.MERGE_AVG, dd.MERGE_RDA, dd.MERGE_RDA, dd.MERGE_AVG]
    M, K = 6, 2
    tokens = rng.integers(1, 1000, size=(len(sizes), M))
    masks = [0b111111, 0b101101, 0b000111, 0b110110]
    host, dev = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 600 + p)
        host.append((theta, v, learners))
        dev.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                        learners=[to_torch_learner(a, "cuda") for a in learners],
                        tokens=[int(t) for t in tokens[p]], quorum_mask=masks[p], K=K, n=n))
    recs_buf = dd.new_records(len(sizes))
    for k in range(2):
        ctx.merge_fragments_batched_rda(dev, M, dd.BF16, ETA, MU, merge_kinds=kinds,
                                        flags=dd.DIAG_STATE, records=recs_buf)
        torch.cuda.synchronize()
        recs = dd.read_records(recs_buf)
        for p, n in enumerate(sizes):
            theta, v, learners = host[p]
            ref = oracle.merge_fragment(theta, v, learners, dev[p]["tokens"], masks[p], K, ETA, MU,
                                        merge=oracle.MERGE_RDA if kinds[p] else oracle.MERGE_AVG)
            assert (recs[p].status, recs[p].idx) == (ref.status, ref.idx)
            assert abs(recs[p].delta_sq - ref.delta_sq) <= TOL_NORM * ref.delta_sq
            assert abs(recs[p].theta_sq - ref.theta_sq) <= TOL_NORM * ref.theta_sq
            assert floor_rel_err(dev[p]["global_"].cpu().numpy(), theta) <= TOL_STATE, (k, p)
            assert floor_rel_err(dev[p]["momentum"].cpu().numpy(), v) <= TOL_STATE, (k, p)
            dev[p]["global_"].copy_(torch.from_numpy(theta))
            dev[p]["momentum"].copy_(torch.from_numpy(v))


@pytest.mark.parametrize("shards", [2, 3])
def test_range_sharded_rda_equals_unsharded(dd, ctx, shards):
    """A fragment cut into element ranges, as a multi-GPU job would hold it: the three passes run
    shard by shard and the hand-over fields of the records are summed in between (here by the
    test, on one GPU, where ranks would all-reduce).  Result: the oracle's merge of the whole
    fragment; whole-fragment diagnostics in every shard's record."""
    from paper_2604_21428_b200 import dist as ddist

    n, M = 300_011, 5
    tokens, mask, K = [100, 200, 0, 400, 500], 0b11101, 2
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 4711)
    o_theta, o_v = theta.copy(), v.copy()
    ref = oracle.merge_fragment(o_theta, o_v, learners, tokens, mask, K, ETA, MU, merge=oracle.MERGE_RDA)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    ranges = [ddist.shard_range(n, r, shards) for r in range(shards)]
    frags = [[dict(global_=t_dev[lo:hi], momentum=v_dev[lo:hi], learners=[t[lo:hi] for t in l_dev],
                   tokens=tokens, quorum_mask=mask, K=K, n=hi - lo)] for lo, hi in ranges]
    recs = [dd.new_records(1) for _ in range(shards)]
    scratch = [torch.empty((hi - lo + 7) // 8 * 8, dtype=torch.float32, device="cuda") for lo, hi in ranges]

    def all_shards_sum(parts):                     # what an all-reduce would leave on every rank
        total = torch.stack(parts).sum(dim=0)
        for p in parts:
            p.copy_(total)

    for p in (dd.RDA_PASS_NORMS, dd.RDA_PASS_DIRECTION, dd.RDA_PASS_APPLY):
        for r in range(shards):
            ctx.merge_fragments_batched_rda_pass(frags[r], M, dd.BF16, ETA, MU, p, records=recs[r],
                                                 scratch=scratch[r], flags=dd.DIAG_STATE)
        torch.cuda.synchronize()
        for name in ddist.RDA_HANDOVER_FIELDS[p]:
            a, b = dd.record_field_columns(name)
            tables = [rec.view(torch.float64).view(-1, dd.RECORD_BYTES // 8) for rec in recs]
            parts = [t[:, a:b].clone() for t in tables]
            all_shards_sum(parts)
            for t, part in zip(tables, parts):
                t[:, a:b] = part
    torch.cuda.synchronize()
    assert floor_rel_err(t_dev.cpu().numpy(), o_theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), o_v) <= TOL_STATE
    for rec in recs:
        _check_record(dd.read_records(rec)[0], ref)


# With at most eight participants the merge takes two launches (Gram matrix of the outer gradients,
# then the ordinary merge with weights derived from it); the cases above with up to eight
# participants ran that form.  The same cases in the three-launch form, which larger participant
# counts and range-sharded fragments use:
@pytest.mark.parametrize("n", [5, 1023, 8192 * 2 + 3, 200_001])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_rda_three_launch_form(dd, ctx, n, dtype):
    _case(dd, ctx, n, 5, dtype, [100, 200, 0, 400, 500], 0b11101, 2, seed=n % 89, three_pass=True)


def test_rda_three_launch_form_special_cases(dd, ctx):
    _case(dd, ctx, 30_000, 4, "f32", [4000, 9000, 100, 2500], 0b1111, 4, seed=5, steps=[4, 3, 1, 5],
          heavy=True, three_pass=True)
    _case(dd, ctx, 30_000, 4, "bf16", [5, 5, 5, 5], 0b1111, 1, seed=6, zero_learner=0, merges=1,
          three_pass=True)
    _case(dd, ctx, 2 * 296 * 8192 + 8192 + 3, 3, "bf16", [700, 0, 900], 0b111, 2, seed=31, merges=1,
          three_pass=True)


def test_rda_two_launch_form_exactly_eight_and_nine_participants(dd, ctx):
    # eight participants: the largest Gram matrix (36 products); nine: the three-launch form takes over
    tokens = [10 * (m + 1) for m in range(12)]
    rec = _case(dd, ctx, 70_001, 12, "bf16", tokens, 0b000011111111, 3, seed=41)
    assert rec.n_part == 8
    rec = _case(dd, ctx, 70_001, 12, "f32", tokens, 0b000011111111, 3, seed=42, merges=1)
    assert rec.n_part == 8
    rec = _case(dd, ctx, 70_001, 12, "bf16", tokens, 0b000111111111, 3, seed=43, merges=1)
    assert rec.n_part == 9
    # one participant: Delta is its own outer gradient
    rec = _case(dd, ctx, 9_001, 3, "bf16", [1, 2, 3], 0b010, 1, seed=44, merges=1)
    assert rec.n_part == 1


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_rda_two_launch_form_around_the_packed_limit(dd, ctx, dtype):
    # up to 6 participants the Gram launch keeps packed even / odd sums, at 7 and 8 scalar ones (another
    # kernel instance): both sides of the limit, several sub-tiles per thread and a ragged end
    tokens = [10 * (m + 1) for m in range(10)]
    for s, seed in ((5, 51), (6, 52), (7, 53)):
        rec = _case(dd, ctx, 3 * 8192 + 1029, 10, dtype, tokens, (1 << s) - 1, 2, seed=seed, merges=1)
        assert rec.n_part == s


def test_rda_two_launch_batch_mixing_participant_counts(dd, ctx):
    # one launch holds fragments on both sides of the packed limit: the launcher takes the instance with
    # the scalar sums for all of them; a second batch of small counts only takes the packed one
    rng = np.random.default_rng(61)
    M, K = 8, 1
    for counts in ([3, 8, 6, 7, 1], [2, 6, 4, 5]):
        sizes = [8192 * 5 + 7 * (p + 1) for p in range(len(counts))]
        tokens = rng.integers(1, 1000, size=(len(sizes), M))
        masks = [(1 << c) - 1 for c in counts]
        host, dev = [], []
        for p, n in enumerate(sizes):
            theta, v, learners = synth.fragment_cpu(n, M, "bf16", 700 + 10 * len(counts) + p)
            host.append((theta, v, learners))
            dev.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                            learners=[to_torch_learner(a, "cuda") for a in learners],
                            tokens=[int(t) for t in tokens[p]], quorum_mask=masks[p], K=K, n=n))
        recs_buf = dd.new_records(len(sizes))
        ctx.merge_fragments_batched_rda(dev, M, dd.BF16, ETA, MU, flags=dd.DIAG_STATE, records=recs_buf)
        torch.cuda.synchronize()
        recs = dd.read_records(recs_buf)
        for p, n in enumerate(sizes):
            theta, v, learners = host[p]
            ref = oracle.merge_fragment(theta, v, learners, dev[p]["tokens"], masks[p], K, ETA, MU,
                                        merge=oracle.MERGE_RDA)
            _check_record(recs[p], ref)
            assert recs[p].n_part == counts[p]
            assert floor_rel_err(dev[p]["global_"].cpu().numpy(), theta) <= TOL_STATE, p
            assert floor_rel_err(dev[p]["momentum"].cpu().numpy(), v) <= TOL_STATE, p


def test_rda_two_launch_form_collinear_gradients(dd, ctx):
    # every learner moved along the same direction by a different amount: the Gram matrix has rank
    # one, a^T G a = (sum a_j k_j)^2 |d|^2, and RDA equals the weighted mean of the gradients
    n, M = 50_000, 4
    rng = np.random.default_rng(5)
    theta = rng.normal(0, 0.02, n).astype(np.float32)
    d = rng.normal(0, 1e-3, n).astype(np.float32)
    learners = [(theta - np.float32(k) * d).astype(np.float32) for k in (1.0, 2.0, 0.5, 4.0)]
    v = np.zeros(n, dtype=np.float32)
    tokens, mask = [3, 1, 4, 1], 0b1111
    o_t, o_v = theta.copy(), v.copy()
    ref = oracle.merge_fragment(o_t, o_v, learners, tokens, mask, 1, ETA, MU, merge=oracle.MERGE_RDA)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    rec_buf = dd.new_records(1)
    ctx.merge_fragment_rda(t_dev, v_dev, [torch.from_numpy(a).cuda() for a in learners], tokens, mask, 1,
                           ETA, MU, flags=dd.DIAG_STATE, record=rec_buf)
    torch.cuda.synchronize()
    _check_record(dd.read_records(rec_buf)[0], ref)
    assert floor_rel_err(t_dev.cpu().numpy(), o_t) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), o_v) <= TOL_STATE


def test_rda_two_launch_bounded_wait_expiry(dd, ctx):
    # the Gram launch stages through CTA-wide barriers of its own: the test hook makes the first
    # stage of every CTA wait for bytes that never come; every wait runs out, the record says so,
    # and the context works normally afterwards
    n, M = 300_000, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 77)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    L = [to_torch_learner(a, "cuda") for a in learners]
    rec_buf = dd.new_records(1)
    ctx.merge_fragment_rda(t_dev, v_dev, L, [1, 2, 3], 0b111, 1, ETA, MU, flags=dd.DEBUG_EXPIRE_WAIT,
                           record=rec_buf)
    torch.cuda.synchronize()
    rec = dd.read_records(rec_buf)[0]
    assert rec.status == dd.STATUS_WAIT_LIMIT and rec.idx == [0, 1, 2]
    t_dev.copy_(torch.from_numpy(theta))
    v_dev.copy_(torch.from_numpy(v))
    ref = oracle.merge_fragment(theta, v, learners, [1, 2, 3], 0b111, 1, ETA, MU, merge=oracle.MERGE_RDA)
    ctx.merge_fragment_rda(t_dev, v_dev, L, [1, 2, 3], 0b111, 1, ETA, MU, flags=dd.DIAG_STATE, record=rec_buf)
    torch.cuda.synchronize()
    _check_record(dd.read_records(rec_buf)[0], ref)
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
