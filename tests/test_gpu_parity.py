"""GPU-vs-oracle parity through the C ABI (element by element, same seeded inputs)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import (TOL_BF16, TOL_STATE, assert_record_matches, bf16_bits_to_f32,
                         floor_rel_err, to_torch_learner)

pytestmark = pytest.mark.gpu

GUARD = 64          # canary elements on both sides of every output buffer
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


def _guarded(host: np.ndarray, dtype, device="cuda", shift=0):
    """Device copy of ``host`` with NaN-free canaries around it; returns (full, view).
    ``shift`` moves the view by that many elements (to leave 32-byte alignment)."""
    n = host.size
    full = torch.full((n + 2 * GUARD,), 12345.0, dtype=dtype, device=device)
    view = full[GUARD + shift:GUARD + shift + n]
    if n:
        view.copy_(torch.from_numpy(host).to(dtype))
    return full, view


def _resync(dev, host):
    """Before the next merge both sides must start from the SAME state: an ulp of
    difference in Theta (6e-8 * 0.1) is of order 1e-5 of the next merge's outer
    gradient, which is a difference of nearly equal numbers.  The oracle's state
    is copied to the device, never the other way round."""
    if host.size:
        dev.copy_(torch.from_numpy(host))


def _check_guard(full, n, shift=0):
    assert torch.all(full[:GUARD + shift] == 12345.0) and \
        torch.all(full[GUARD + shift + n:] == 12345.0), "write outside the output buffer"


def run_case(dd, ctx, n, M, dtype, tokens, mask, K, *, seed=0, steps=None, flags=0, merges=2,
             use_out=True, poison_absent=False, null_absent=False, eta=ETA, mu=MU, shift=0):
    theta, v, learners = synth.fragment_cpu(n, M, dtype, seed)
    part = [m for m in range(M) if (mask >> m) & 1 and tokens[m] > 0]
    if poison_absent:
        for m in range(M):
            if m not in part:
                learners[m] = np.full_like(learners[m], 0x7fc0 if dtype == "bf16" else np.nan)
    o_learners = list(learners)
    if null_absent:
        o_learners = [a if m in part else None for m, a in enumerate(learners)]
    d_learners = [to_torch_learner(a, "cuda") for a in o_learners]
    t_full, t_dev = _guarded(theta, torch.float32, shift=shift)
    v_full, v_dev = _guarded(v, torch.float32)
    out_full = out_dev = None
    if use_out:
        out_full, out_dev = _guarded(np.zeros(n, dtype=np.float32), torch.bfloat16)
    rec_buf = dd.new_records(1)
    heavy = bool(flags & dd.HEAVY_BALL)
    for k in range(merges):
        o_out = np.zeros(n, dtype=np.uint16) if use_out else None
        ref = oracle.merge_fragment(theta, v, o_learners, tokens, mask, K, eta, mu, steps=steps,
                                    nesterov=not heavy, out_bf16=o_out)
        ctx.merge_fragment(t_dev, v_dev, d_learners, tokens, mask, K, eta, mu, n=n,
                           learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32, steps=steps,
                           flags=flags, out_bf16=out_dev, record=rec_buf)
        torch.cuda.synchronize()
        got = dd.read_records(rec_buf)[0]
        assert_record_matches(got, ref, diag_state=bool(flags & dd.DIAG_STATE),
                              per_learner=bool(flags & dd.DIAG_PER_LEARNER))
        e_t = floor_rel_err(t_dev.cpu().numpy(), theta)
        e_v = floor_rel_err(v_dev.cpu().numpy(), v)
        assert e_t <= TOL_STATE and e_v <= TOL_STATE, (k, e_t, e_v)
        if use_out and ref.status == 0:
            e_o = floor_rel_err(bf16_bits_to_f32(out_dev), oracle.bf16_to_f32(o_out))
            assert e_o <= TOL_BF16, e_o
            # identical except where the fp32 state differs by an ulp across a rounding boundary
            same = np.mean(out_dev.cpu().view(torch.int16).numpy().view(np.uint16) == o_out) if n else 1.0
            assert same > 0.999
        _check_guard(t_full, n, shift)
        _check_guard(v_full, n)
        if use_out:
            _check_guard(out_full, n)
        if ref.status != 0 and use_out:
            assert torch.all(out_dev == 0)
        _resync(t_dev, theta)
        _resync(v_dev, v)
    return got


def test_tiny_config(dd, ctx):
    w = synth.workload("tiny")
    run_case(dd, ctx, w.fragment_sizes[0], w.M, "f32", w.tokens[0].tolist(), w.masks[0], w.K,
             seed=w.seed, flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER)


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 1023, 8192, 8193, 3 * 8192 + 5, (1 << 20) + 3])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_ragged_sizes(dd, ctx, n, dtype):
    run_case(dd, ctx, n, 5, dtype, [100, 200, 0, 400, 500], 0b11101, 2, seed=n % 97,
             flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_state_only_16_byte_aligned(dd, ctx, dtype):
    # Theta 16- but not 32-byte aligned: the 2 x 128-bit access path instead of 256-bit
    run_case(dd, ctx, 40_003, 5, dtype, [100, 200, 0, 400, 500], 0b11101, 2, seed=31,
             flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, shift=4)
    run_case(dd, ctx, 40_003, 5, dtype, [100, 200, 0, 400, 500], 0b11101, 2, seed=31, flags=0,
             shift=4)


@pytest.mark.parametrize("flags", [0, 1, 2, 4, 7])
def test_flag_combinations(dd, ctx, flags):
    run_case(dd, ctx, 50_000, 8, "bf16", [5, 6, 7, 8, 9, 10, 11, 12], 0b10110111, 3, seed=3,
             flags=flags, merges=3)


def test_no_record_no_output(dd, ctx):
    n, M = 40_000, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 5)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    d_learners = [to_torch_learner(a, "cuda") for a in learners]
    oracle.merge_fragment(theta, v, learners, [1, 2, 3], 0b111, 1, ETA, MU)
    ctx.merge_fragment(t_dev, v_dev, d_learners, [1, 2, 3], 0b111, 1, ETA, MU)
    torch.cuda.synchronize()
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE


def test_dense150m_shape_scaled(dd, ctx):
    # the 8-learner / 6-participant bf16 workload, one fragment at 1/400 of its size
    w = synth.workload("dense150m")
    n = w.fragment_sizes[0] // 400 + 3
    rec = run_case(dd, ctx, n, w.M, "bf16", w.tokens[0].tolist(), w.masks[0], w.K, seed=w.seed,
                   flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, poison_absent=True)
    assert rec.n_part == 6


def test_scale_shape_scaled(dd, ctx):
    # 32 learners, 24 participants (the steady-state workload) at reduced n
    w = synth.workload("scale500m")
    rec = run_case(dd, ctx, 300_007, w.M, "bf16", w.tokens[0].tolist(), w.masks[0], w.K,
                   seed=w.seed, flags=dd.DIAG_STATE, null_absent=True)
    assert rec.n_part == 24


@pytest.mark.parametrize("dtype,flags", [("bf16", 4), ("f32", 4 | 2)])
def test_several_tiles_per_cta_element_by_element(dd, ctx, dtype, flags):
    # 2 x 296 CTAs' worth of 8192-element tiles plus a ragged rest: every CTA of the persistent
    # grid walks more than one tile and its ring wraps many times; checked on every element
    n = 2 * 296 * 8192 + 3 * 8192 + 5
    run_case(dd, ctx, n, 3, dtype, [700, 0, 900], 0b111, 2, seed=77, flags=flags, merges=1)


def test_batched_large_fragments_element_by_element(dd, ctx):
    # CTAs cross fragment boundaries in mid-stream: tile counts that are not multiples of the grid
    sizes = [3_000_017, 1_500_001, 8, 2_000_003]
    M = 3
    tokens = np.array([[5, 7, 9], [1, 0, 4], [3, 3, 3], [9, 8, 0]])
    _batched_case(dd, ctx, sizes, M, "bf16", tokens, [0b111, 0b101, 0b110, 0b011], 2, seed=21,
                  flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, merges=1)


def test_batched_ring_depth_changes_between_fragments(dd, ctx):
    # the staging ring runs shallower below 8 bf16 participants: fragments on either side of that
    # count alternate, about 100 tiles each, so that most CTAs switch depth between their tiles
    M = 12
    counts = [3, 9, 7, 8, 12, 1, 10, 5]
    sizes = [8192 * 100 + 17 * (p + 1) for p in range(len(counts))]
    rng = np.random.default_rng(33)
    tokens = rng.integers(1, 1000, size=(len(sizes), M))
    masks = []
    for c in counts:
        chosen = rng.choice(M, size=c, replace=False)
        masks.append(int(sum(1 << int(m) for m in chosen)))
    recs = _batched_case(dd, ctx, sizes, M, "bf16", tokens, masks, 1, seed=34,
                         flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER)
    assert [r.n_part for r in recs] == counts


def test_masked_learners_are_never_read(dd, ctx):
    # absent learners: NaN payloads, then null pointers
    run_case(dd, ctx, 20_001, 6, "bf16", [9, 9, 0, 9, 9, 9], 0b101011, 2, seed=8, poison_absent=True)
    run_case(dd, ctx, 20_001, 6, "f32", [9, 9, 0, 9, 9, 9], 0b101011, 2, seed=8, null_absent=True)


def test_single_learner_and_sixty_four(dd, ctx):
    run_case(dd, ctx, 10_000, 1, "bf16", [7], 1, 1, seed=1, flags=6)
    tokens = list(range(1, 65))
    run_case(dd, ctx, 9_001, 64, "bf16", tokens, (1 << 64) - 1, 64, seed=2, flags=6, merges=1)
    rec = run_case(dd, ctx, 9_001, 64, "bf16", tokens, 1 << 63, 1, seed=2, flags=6, merges=1,
                   null_absent=True)
    assert rec.idx == [63]
    tokens[40] = 0
    rec = run_case(dd, ctx, 9_001, 64, "f32", tokens, ((1 << 64) - 1) ^ (1 << 5), 10, seed=2,
                   flags=6, merges=1)
    assert rec.n_part == 62 and 40 not in rec.idx and 5 not in rec.idx


def test_quorum_not_met_and_zero_tokens(dd, ctx):
    rec = run_case(dd, ctx, 5_000, 4, "bf16", [1, 2, 3, 4], 0b0011, 3, seed=4)
    assert rec.status == dd.STATUS_QUORUM_NOT_MET and rec.n_part == 2
    rec = run_case(dd, ctx, 5_000, 4, "bf16", [0, 0, 0, 0], 0b1111, 0, seed=4)
    assert rec.status == dd.STATUS_QUORUM_NOT_MET and rec.n_part == 0


def test_huge_token_counts(dd, ctx):
    run_case(dd, ctx, 9_000, 3, "bf16", [2**62, 2**61, 2**61 + 12345], 0b111, 3, seed=44, merges=1)
    run_case(dd, ctx, 9_000, 3, "bf16", [2**40, 2**45, 2**50 + 1], 0b111, 3, seed=45, merges=1,
             steps=[3, 2**20, 7])


def test_steps_weighting(dd, ctx):
    tokens = [40960, 8192, 123456, 99999, 5]
    steps = [10, 1, 33, 7, 5]
    rec = run_case(dd, ctx, 30_011, 5, "bf16", tokens, 0b11111, 5, seed=6, steps=steps, flags=6)
    raw = [t * (t / s) for t, s in zip(tokens, steps)]
    assert math.isclose(rec.w_total, sum(raw), rel_tol=1e-12)


def test_lr1_mu0_gives_weighted_mean(dd, ctx):
    run_case(dd, ctx, 12_345, 4, "f32", [1000, 3000, 2000, 500], 0b1111, 4, seed=7, eta=1.0, mu=0.0,
             merges=1)        # a second merge would have Delta == rounding noise only


def test_nan_in_participant_propagates(dd, ctx):
    n, M = 4_096 + 17, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 12)
    learners[1][100] = 0x7fc0          # NaN
    learners[2][200] = 0x7f80          # +Inf
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    d_learners = [to_torch_learner(a, "cuda") for a in learners]
    oracle.merge_fragment(theta, v, learners, [1, 2, 3], 0b111, 1, ETA, MU)
    ctx.merge_fragment(t_dev, v_dev, d_learners, [1, 2, 3], 0b111, 1, ETA, MU)
    torch.cuda.synchronize()
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
    assert np.isnan(theta[100]) and np.isinf(theta[200])


def _batched_case(dd, ctx, sizes, M, dtype, tokens, masks, K, *, seed, flags, steps=None,
                  merges=2):
    P = len(sizes)
    host, dev = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, dtype, seed * 1000 + p)
        part = [m for m in range(M) if (masks[p] >> m) & 1 and int(tokens[p][m]) > 0]
        o_learners = [a if m in part else None for m, a in enumerate(learners)]
        host.append((theta, v, o_learners))
        t_full, t_dev = _guarded(theta, torch.float32)
        v_full, v_dev = _guarded(v, torch.float32)
        o_full, o_dev = _guarded(np.zeros(n, dtype=np.float32), torch.bfloat16)
        dev.append(dict(t_full=t_full, v_full=v_full, o_full=o_full, global_=t_dev, momentum=v_dev,
                        out_bf16=o_dev, learners=[to_torch_learner(a, "cuda") for a in o_learners],
                        tokens=[int(x) for x in tokens[p]], quorum_mask=masks[p], K=K, n=n,
                        steps=None if steps is None else [int(x) for x in steps[p]]))
    rec_buf = dd.new_records(P)
    heavy = bool(flags & dd.HEAVY_BALL)
    for k in range(merges):
        ctx.merge_fragments_batched(dev, M, dd.BF16 if dtype == "bf16" else dd.F32, ETA, MU,
                                    flags=flags, records=rec_buf)
        torch.cuda.synchronize()
        recs = dd.read_records(rec_buf)
        for p, n in enumerate(sizes):
            theta, v, o_learners = host[p]
            o_out = np.zeros(n, dtype=np.uint16)
            ref = oracle.merge_fragment(theta, v, o_learners, dev[p]["tokens"], masks[p], K, ETA,
                                        MU, steps=dev[p]["steps"], nesterov=not heavy,
                                        out_bf16=o_out)
            assert_record_matches(recs[p], ref, diag_state=bool(flags & dd.DIAG_STATE),
                                  per_learner=bool(flags & dd.DIAG_PER_LEARNER))
            assert floor_rel_err(dev[p]["global_"].cpu().numpy(), theta) <= TOL_STATE, (k, p)
            assert floor_rel_err(dev[p]["momentum"].cpu().numpy(), v) <= TOL_STATE, (k, p)
            if ref.status == 0:
                assert floor_rel_err(bf16_bits_to_f32(dev[p]["out_bf16"]),
                                     oracle.bf16_to_f32(o_out)) <= TOL_BF16
            for key in ("t_full", "v_full", "o_full"):
                _check_guard(dev[p][key], n)
            _resync(dev[p]["global_"], theta)
            _resync(dev[p]["momentum"], v)
    return recs


def test_batched_ragged_mixed_status(dd, ctx):
    rng = np.random.default_rng(5)
    sizes = [8192 * 3 + 1, 0, 17, 100_000, 8192, 250_003, 5]
    M = 6
    tokens = rng.integers(0, 50, size=(len(sizes), M))
    masks = [int(rng.integers(1, 1 << M)) for _ in sizes]
    masks[3] = 0b000011                  # 2 participants at most: below K = 3
    tokens[3] = [5, 5, 5, 5, 5, 5]
    recs = _batched_case(dd, ctx, sizes, M, "bf16", tokens, masks, 3, seed=9,
                         flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER)
    assert recs[3].status == dd.STATUS_QUORUM_NOT_MET
    assert any(r.status == 0 for r in recs)


def test_batched_many_small_fragments(dd, ctx):
    # more fragments than CTAs can each own: every CTA walks across several fragments
    rng = np.random.default_rng(6)
    P, M = 700, 4
    sizes = [int(x) for x in rng.integers(1, 3000, size=P)]
    tokens = rng.integers(1, 1000, size=(P, M))
    steps = rng.integers(1, 9, size=(P, M))
    masks = [int(rng.integers(1, 1 << M)) for _ in range(P)]
    _batched_case(dd, ctx, sizes, M, "f32", tokens, masks, 1, seed=10, flags=dd.DIAG_STATE,
                  steps=steps, merges=1)


@pytest.mark.parametrize("name,factor", [("dense150m", 1 / 256), ("dense1b3", 1 / 2048),
                                         ("moe4b", 1 / 4096)])
def test_batched_workload_shapes_scaled(dd, ctx, name, factor):
    w = synth.scaled(synth.workload(name), factor)
    recs = _batched_case(dd, ctx, w.fragment_sizes, w.M, "bf16", w.tokens, w.masks, w.K,
                         seed=w.seed, flags=dd.DIAG_STATE, merges=2)
    for p, r in enumerate(recs):
        assert r.status == 0 and r.n_part == sum(1 for m in range(w.M) if (w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0)


def test_back_to_back_calls_share_context(dd, ctx):
    # many launches without host synchronisation in between (staging ring, tickets re-armed)
    n, M = 70_001, 4
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 21)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    d_learners = [to_torch_learner(a, "cuda") for a in learners]
    rec_buf = dd.new_records(1)
    frag = dict(global_=t_dev, momentum=v_dev, learners=d_learners, tokens=[4, 3, 2, 1],
                quorum_mask=0b1111, K=4, n=n)
    for k in range(12):
        if k % 2:
            ctx.merge_fragment(t_dev, v_dev, d_learners, [4, 3, 2, 1], 0b1111, 4, ETA, MU,
                               flags=dd.DIAG_STATE, record=rec_buf)
        else:
            ctx.merge_fragments_batched([frag], M, dd.BF16, ETA, MU, flags=dd.DIAG_STATE,
                                        records=rec_buf)
        ref = oracle.merge_fragment(theta, v, learners, [4, 3, 2, 1], 0b1111, 4, ETA, MU)
    torch.cuda.synchronize()
    # 12 merges without resynchronising the state: rounding differences of Theta
    # feed back through the near-cancelling outer gradient, so only a loose
    # agreement is expected here; this test is about the launch machinery.
    # (With fixed learners the momentum decays towards 0, so it is compared absolutely.)
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= 1e-4
    assert float(np.max(np.abs(v_dev.cpu().numpy() - v))) <= 1e-7
    got = dd.read_records(rec_buf)[0]
    assert got.status == 0 and got.idx == ref.idx
    assert got.w_hat == [float(np.float32(w)) for w in ref.w_hat]


def test_argument_validation(dd, ctx):
    n, M = 1024, 3
    t = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    L = [torch.zeros(n, device="cuda", dtype=torch.bfloat16) for _ in range(M)]

    def rc_of(fn):
        with pytest.raises(dd.DDMergeError) as e:
            fn()
        return e.value.rc

    good = dict(n=n, learner_dtype=dd.BF16)
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, 4, ETA, MU, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, -1, ETA, MU, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, 1, float("nan"), MU, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, 1, ETA, float("inf"), **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, [L[0], None, L[2]], [1, 1, 1], 7, 1, ETA, MU, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, 1, ETA, MU, steps=[1, 0, 1], **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [1, 1, 1], 7, 1, ETA, MU, flags=1 << 9, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t, v, L, [2**63, 2**63, 1], 7, 1, ETA, MU, **good)) == dd.ERR_INVALID_ARG
    assert rc_of(lambda: ctx.merge_fragment(t.data_ptr() + 4, v, L, [1, 1, 1], 7, 1, ETA, MU, n=n - 8, learner_dtype=dd.BF16)) == dd.ERR_ALIGNMENT
    assert rc_of(lambda: ctx.merge_fragment(t, v, [L[0], L[1].data_ptr() + 2, L[2]], [1, 1, 1], 7, 1, ETA, MU, n=n - 8, learner_dtype=dd.BF16)) == dd.ERR_ALIGNMENT
    assert rc_of(lambda: ctx.merge_fragment(t, t, L, [1, 1, 1], 7, 1, ETA, MU, **good)) == dd.ERR_ALIAS
    assert rc_of(lambda: ctx.merge_fragment(t, v, [L[0], t, L[2]], [1, 1, 1], 7, 1, ETA, MU, **good)) == dd.ERR_ALIAS
    assert rc_of(lambda: ctx.merge_fragment(t, v, L * 22, [1] * 66, 7, 1, ETA, MU, **good)) == dd.ERR_TOO_MANY_LEARNERS
    # an absent learner may alias anything or be null: it is never touched
    ctx.merge_fragment(t, v, [L[0], t, None], [1, 1, 1], 0b001, 1, ETA, MU, **good)
    # the same learner buffer listed twice simply counts twice
    ctx.merge_fragment(t, v, [L[0], L[0], L[1]], [1, 1, 1], 7, 1, ETA, MU, **good)
    torch.cuda.synchronize()


# (2_500_003, 0): the default chunk is 2^20 elements there, so three chunks with a ragged last one
@pytest.mark.parametrize("n,chunk", [(100_003, 8192), (50_000, 0), (7, 8), (0, 0), (65_536, 16_384), (2_500_003, 0)])
def test_host_buffers_entry_point(dd, ctx, n, chunk):
    # operands in (pinned) host memory, pipelined through the GPU in chunks
    M = 6
    tokens, mask, K = [10, 0, 30, 40, 50, 60], 0b111101, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 77)
    part = [0, 2, 3, 4, 5]
    h_theta = torch.from_numpy(theta.copy()).pin_memory()
    h_v = torch.from_numpy(v.copy()).pin_memory()
    h_out = torch.zeros(n, dtype=torch.bfloat16).pin_memory()
    h_learners = [to_torch_learner(a, "cpu").pin_memory() if m in part else None
                  for m, a in enumerate(learners)]
    o_learners = [a if m in part else None for m, a in enumerate(learners)]
    for k in range(2):
        o_out = np.zeros(n, dtype=np.uint16)
        ref = oracle.merge_fragment(theta, v, o_learners, tokens, mask, K, ETA, MU, out_bf16=o_out)
        got = ctx.merge_fragment_host(h_theta, h_v, h_learners, tokens, mask, K, ETA, MU, n=n,
                                      learner_dtype=dd.BF16, flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER,
                                      out_bf16=h_out, chunk_elems=chunk)
        assert_record_matches(got, ref)
        assert floor_rel_err(h_theta.numpy(), theta) <= TOL_STATE
        assert floor_rel_err(h_v.numpy(), v) <= TOL_STATE
        assert floor_rel_err(bf16_bits_to_f32(h_out), oracle.bf16_to_f32(o_out)) <= TOL_BF16
        if n:
            h_theta.copy_(torch.from_numpy(theta))
            h_v.copy_(torch.from_numpy(v))
    # quorum not met: nothing is transferred or written
    before = h_theta.clone()
    got = ctx.merge_fragment_host(h_theta, h_v, h_learners, tokens, mask, 6, ETA, MU, n=n,
                                  learner_dtype=dd.BF16)
    assert got.status == dd.STATUS_QUORUM_NOT_MET and got.n_part == 5
    assert torch.equal(before, h_theta)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("alpha,shift", [(0.0, 0), (0.0, 8), (0.5, 0), (0.25, 8)])
def test_broadcast_to_learners(dd, ctx, dtype, alpha, shift):
    # learner side of an update: theta_m <- alpha theta_m + (1 - alpha) Theta'; copies that start
    # on a 32-byte boundary (shift 0) take 32-byte stores, copies 16 bytes off it (shift 8) do not
    n, M = 50_003, 5
    theta, _, learners = synth.fragment_cpu(n, M, dtype, 91)
    mask = 0b10110
    t_dev = torch.from_numpy(theta).cuda()
    full = [_guarded(a.view(np.int16) if dtype == "bf16" else a,
                     torch.int16 if dtype == "bf16" else torch.float32,
                     shift=shift if dtype == "bf16" else shift // 2) for a in learners]
    views = [v.view(torch.bfloat16) if dtype == "bf16" else v for _, v in full]
    ptrs = [views[m] if m != 0 else None for m in range(M)]          # learner 0: not selected, null
    ctx.broadcast_fragment(t_dev, ptrs, mask, alpha, n=n, learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32)
    torch.cuda.synchronize()
    for m in range(M):
        got = views[m].cpu()
        got = got.view(torch.int16).numpy().view(np.uint16) if dtype == "bf16" else got.numpy()
        ref = learners[m].copy()
        if (mask >> m) & 1:
            oracle.apply_to_learner(ref, theta, alpha)
            if alpha == 0.0:
                np.testing.assert_array_equal(got, ref)
            elif dtype == "bf16":
                assert floor_rel_err(oracle.bf16_to_f32(got), oracle.bf16_to_f32(ref)) <= TOL_BF16
                assert np.mean(got == ref) > 0.999
            else:
                assert floor_rel_err(got, ref) <= 1e-6
        else:
            np.testing.assert_array_equal(got, ref)                # untouched
        _check_guard(full[m][0].float(), n, shift if dtype == "bf16" else shift // 2)


def test_bounded_wait_expires_and_context_survives(dd, ctx):
    # Error path of the staged kernel: with the test hook every warp's first copy waits
    # for bytes that never come; the bounded wait gives up after about a second, the
    # record says so, nothing hangs, and the same context merges correctly afterwards.
    n, M = 20_000, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 61)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    L = [to_torch_learner(a, "cuda") for a in learners]
    rec_buf = dd.new_records(1)
    ctx.merge_fragment(t_dev, v_dev, L, [1, 2, 3], 0b111, 1, ETA, MU, flags=dd.DEBUG_EXPIRE_WAIT,
                       record=rec_buf)
    torch.cuda.synchronize()
    rec = dd.read_records(rec_buf)[0]
    assert rec.status == dd.STATUS_WAIT_LIMIT and rec.idx == [0, 1, 2]
    # the context and the device are still healthy: a normal merge matches the oracle
    t_dev.copy_(torch.from_numpy(theta))
    v_dev.copy_(torch.from_numpy(v))
    ref = oracle.merge_fragment(theta, v, learners, [1, 2, 3], 0b111, 1, ETA, MU)
    ctx.merge_fragment(t_dev, v_dev, L, [1, 2, 3], 0b111, 1, ETA, MU, flags=dd.DIAG_STATE,
                       record=rec_buf)
    torch.cuda.synchronize()
    assert_record_matches(dd.read_records(rec_buf)[0], ref, per_learner=False)
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE


def test_bounded_wait_expiry_marks_every_incomplete_fragment_of_a_batch(dd, ctx):
    # Five fragments of 100 tiles on a grid of at most 296 CTAs: most CTAs own tiles of two
    # fragments.  With the hook every warp gives up in the first fragment it works on and skips
    # its rows of the later ones, so every fragment is incomplete and must say so (a fragment
    # left at status 0 would present partial norms as valid).
    grid, _, tile = ctx.launch_geometry(dd.BF16)
    P, M, n = 5, 3, 100 * tile
    assert P * 100 > grid
    frags, hosts = [], []
    for p in range(P):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 70 + p)
        hosts.append((theta, v, learners))
        frags.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                          learners=[to_torch_learner(a, "cuda") for a in learners],
                          tokens=[1 + p, 2, 3], quorum_mask=0b111, K=1, n=n))
    rec_buf = dd.new_records(P)
    ctx.merge_fragments_batched(frags, M, dd.BF16, ETA, MU, flags=dd.DEBUG_EXPIRE_WAIT, records=rec_buf)
    torch.cuda.synchronize()
    recs = dd.read_records(rec_buf)
    assert [r.status for r in recs] == [dd.STATUS_WAIT_LIMIT] * P
    assert all(r.idx == [0, 1, 2] for r in recs)
    # the next call on the same context and records is a normal merge again
    for f, (theta, v, _) in zip(frags, hosts):
        f["global_"].copy_(torch.from_numpy(theta))
        f["momentum"].copy_(torch.from_numpy(v))
    ctx.merge_fragments_batched(frags, M, dd.BF16, ETA, MU, flags=dd.DIAG_STATE, records=rec_buf)
    torch.cuda.synchronize()
    for p, (rec, f, (theta, v, learners)) in enumerate(zip(dd.read_records(rec_buf), frags, hosts)):
        ref = oracle.merge_fragment(theta, v, learners, [1 + p, 2, 3], 0b111, 1, ETA, MU)
        assert_record_matches(rec, ref, per_learner=False)
        assert floor_rel_err(f["global_"].cpu().numpy(), theta) <= TOL_STATE
        assert floor_rel_err(f["momentum"].cpu().numpy(), v) <= TOL_STATE


def test_hand_worked_example_on_gpu(dd, ctx):
    # the two-learner merge worked on paper in tests/golden/merge_hand_worked.txt; every
    # intermediate is exact in binary32, so the GPU must reproduce it bit for bit
    import os
    g = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "merge_hand_worked.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            key, *vals = line.split()
            g[key] = [float(x) for x in vals]
    for flags, key in ((0, "theta_nesterov"), (dd.HEAVY_BALL, "theta_heavy")):
        t = torch.tensor(g["theta"], dtype=torch.float32, device="cuda")
        v = torch.tensor(g["momentum"], dtype=torch.float32, device="cuda")
        L = [torch.tensor(g["learner0"], dtype=torch.float32, device="cuda"),
             torch.tensor(g["learner1"], dtype=torch.float32, device="cuda")]
        rec_buf = dd.new_records(1)
        ctx.merge_fragment(t, v, L, [int(x) for x in g["tokens"]], 0b11, 2, g["eta"][0], g["mu"][0],
                           flags=flags | dd.DIAG_PER_LEARNER, record=rec_buf)
        torch.cuda.synchronize()
        rec = dd.read_records(rec_buf)[0]
        assert rec.w_hat == g["w_hat"] and rec.delta_sq == g["delta_sq"][0]
        assert rec.delta_m_sq == g["delta_m_sq"]
        assert v.cpu().tolist() == g["momentum_new"] and t.cpu().tolist() == g[key]


def test_participation_and_weights_random_sweep(dd, ctx):
    # 300 random (M, mask, tokens, steps, K): participant set, order, status bit-exact;
    # weights bit-exact as float32 without steps, to 1 ulp-ish with steps (fp64 sum order is fixed)
    rng = np.random.default_rng(2024)
    n = 64
    theta = torch.zeros(n, device="cuda")
    mom = torch.zeros(n, device="cuda")
    pool = [torch.full((n,), 0.01 * (m + 1), device="cuda", dtype=torch.bfloat16) for m in range(64)]
    rec_buf = dd.new_records(1)
    for trial in range(300):
        M = int(rng.integers(1, 65))
        tokens = [int(t) for t in rng.integers(0, 4, size=M) * rng.integers(1, 10**6, size=M)]
        mask = int(rng.integers(0, 1 << 62)) | (int(rng.integers(0, 4)) << 62)
        K = int(rng.integers(0, M + 1))
        steps = None if trial % 2 else [int(x) for x in rng.integers(1, 1000, size=M)]
        st, idx = oracle.participants(mask, tokens, K)
        ctx.merge_fragment(theta, mom, pool[:M], tokens, mask, K, ETA, MU, n=n, learner_dtype=dd.BF16,
                           steps=steps, record=rec_buf)
        torch.cuda.synchronize()
        rec = dd.read_records(rec_buf)[0]
        assert (rec.status, rec.idx) == (st, idx), (trial, M, K)
        if st == 0:
            _, w_hat, W = oracle.weights(tokens, steps, idx)
            assert rec.w_hat == [float(np.float32(w)) for w in w_hat], trial
            assert abs(rec.w_total - W) <= 1e-15 * W


def test_two_contexts_on_two_streams(dd):
    # Separate contexts own separate workspaces, so their launches may overlap on the GPU.
    n, M = 400_003, 4
    results = []
    ctxs = [dd.Context(0), dd.Context(0)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    cases = []
    for i in range(2):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 300 + i)
        cases.append((theta, v, learners, torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda(),
                      [to_torch_learner(a, "cuda") for a in learners], dd.new_records(1)))
    torch.cuda.synchronize()
    for rep in range(3):
        for i in range(2):
            theta, v, learners, t_dev, v_dev, L, rec = cases[i]
            ctxs[i].merge_fragment(t_dev, v_dev, L, [3, 1, 4, 1 + i], 0b1111, 2, ETA, MU,
                                   flags=dd.DIAG_STATE, record=rec, stream=streams[i])
    torch.cuda.synchronize()
    for i in range(2):
        theta, v, learners, t_dev, v_dev, L, rec = cases[i]
        for rep in range(3):
            ref = oracle.merge_fragment(theta, v, learners, [3, 1, 4, 1 + i], 0b1111, 2, ETA, MU)
        got = dd.read_records(rec)[0]
        assert got.status == 0 and got.idx == ref.idx
        assert floor_rel_err(t_dev.cpu().numpy(), theta) <= 1e-4        # three merges without resync
        assert float(np.max(np.abs(v_dev.cpu().numpy() - v))) <= 1e-7
        assert abs(got.theta_sq - ref.theta_sq) <= 1e-4 * ref.theta_sq
    for c in ctxs:
        c.close()


def test_random_shape_sweep(dd, ctx):
    # 60 random (n, M, participants, dtype, alignment, flags, steps, output) combinations
    rng = np.random.default_rng(77)
    for trial in range(60):
        n = int(rng.choice([rng.integers(1, 300), rng.integers(300, 9000), rng.integers(9000, 70000)]))
        M = int(rng.integers(1, 13))
        tokens = [int(t) for t in rng.integers(0, 3, size=M) * rng.integers(1, 5000, size=M)]
        mask = int(rng.integers(0, 1 << M))
        K = int(rng.integers(0, M + 1))
        dtype = "bf16" if rng.random() < 0.6 else "f32"
        flags = int(rng.choice([0, 1, 2, 4, 6, 7]))
        steps = None if rng.random() < 0.5 else [int(x) for x in rng.integers(1, 50, size=M)]
        run_case(dd, ctx, n, M, dtype, tokens, mask, K, seed=1000 + trial, steps=steps, flags=flags,
                 merges=1, use_out=bool(rng.random() < 0.5), null_absent=bool(rng.random() < 0.5),
                 shift=int(rng.choice([0, 4])))


def test_cuda_graph_capture_and_replay(dd, ctx):
    """The single-fragment call is capture-safe once the context has its workspace: captured into a
    CUDA graph and replayed, it gives the oracle's result, replay after replay."""
    n, M = 40_003, 4
    tokens, mask, K = [5, 0, 7, 9], 0b1101, 2
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 321)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    rec_buf = dd.new_records(1)
    ctx.merge_fragment(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU, flags=dd.DIAG_STATE, record=rec_buf)
    torch.cuda.synchronize()                                 # workspace exists from here on
    ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, ETA, MU)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            ctx.merge_fragment(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU, flags=dd.DIAG_STATE,
                               record=rec_buf, stream=side)
    for _ in range(3):
        t_dev.copy_(torch.from_numpy(synth.fragment_cpu(n, M, "bf16", 321)[0]))
        v_dev.zero_()
        rec_buf.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got = dd.read_records(rec_buf)[0]
        assert_record_matches(got, ref, diag_state=True, per_learner=False)
        assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
        assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE


def test_prepared_call_equals_plain_call(dd, ctx):
    # arguments marshalled once, the mask given per call, token counts updated in place in between:
    # bit-identical to the ordinary call on the same inputs
    n, M = 50_003, 5
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 123)
    a = [torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()]
    b = [torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()]
    l_dev = [to_torch_learner(x, "cuda") for x in learners]
    rec_a, rec_b = dd.new_records(1), dd.new_records(1)
    tokens = dd.pack_u64([10, 20, 30, 40, 50])
    call = ctx.prepare_merge_fragment(a[0], a[1], l_dev, tokens, 2, ETA, MU, flags=dd.DIAG_STATE, record=rec_a)
    for mask, new_tokens in ((0b10111, [10, 20, 30, 40, 50]), (0b01110, [5, 0, 7, 9, 11]), (0b00001, [1, 1, 1, 1, 1])):
        for m, t in enumerate(new_tokens):
            tokens[m] = t
        call(mask)
        ctx.merge_fragment(b[0], b[1], l_dev, new_tokens, mask, 2, ETA, MU, flags=dd.DIAG_STATE, record=rec_b)
        torch.cuda.synchronize()
        ra, rb = dd.read_records(rec_a)[0], dd.read_records(rec_b)[0]
        assert (ra.status, ra.idx, ra.w_hat, ra.delta_sq) == (rb.status, rb.idx, rb.w_hat, rb.delta_sq)
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert dd.read_records(rec_a)[0].status == dd.STATUS_QUORUM_NOT_MET      # one participant, K = 2


def test_packed_pointer_and_count_arrays(dd, ctx):
    """Pre-marshalled learner addresses and token counts give the same merge as lists."""
    n, M = 20_001, 5
    tokens, mask, K = [3, 0, 8, 1, 6], 0b11101, 2
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 55)
    ref = oracle.merge_fragment(theta.copy(), v.copy(), learners, tokens, mask, K, ETA, MU)
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    results = []
    for packed in (False, True):
        t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
        rec_buf = dd.new_records(1)
        ls = dd.pack_pointers(l_dev) if packed else l_dev
        tk = dd.pack_u64(tokens) if packed else tokens
        ctx.merge_fragment(t_dev, v_dev, ls, tk, mask, K, ETA, MU, n=n, learner_dtype=dd.BF16,
                           flags=dd.DIAG_STATE, record=rec_buf)
        torch.cuda.synchronize()
        results.append((t_dev.cpu(), v_dev.cpu(), dd.read_records(rec_buf)[0]))
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])
    assert results[0][2].idx == results[1][2].idx == ref.idx
    with pytest.raises(ValueError):
        ctx.merge_fragment(results[0][0].cuda(), results[0][1].cuda(), dd.pack_pointers(l_dev), tokens,
                           mask, K, ETA, MU, n=n)


def test_bitwise_reproducible_run_to_run(dd, ctx):
    """Same inputs, same bits: every element has one owner and the norms are reduced in a fixed
    order (per-CTA partials added by the last CTA in CTA order), whatever the CTA timing."""
    n, M = 2 * 296 * 8192 + 4099, 6
    tokens, mask, K = [11, 7, 0, 5, 9, 13], 0b111011, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 404)
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    first = None
    for rep in range(12):
        t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
        out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        rec_buf = dd.new_records(1)
        ctx.merge_fragment(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU,
                           flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, out_bf16=out, record=rec_buf)
        torch.cuda.synchronize()
        got = (t_dev, v_dev, out.view(torch.int16), rec_buf.clone())
        if first is None:
            first = got
        else:
            assert all(torch.equal(a, b) for a, b in zip(first, got)), rep


@pytest.mark.parametrize("kind,s,k", [("avg", 9, 0), ("push", 8, 8), ("push", 8, 1), ("rda", 6, 0), ("rda", 8, 0)])
def test_bitwise_reproducible_over_repeated_merges(dd, ctx, kind, s, k):
    """Twenty merges in a row from the same start, twice: the same bits at the end, for the launch
    shapes that differ from the plain merge's (full ring at 9 participants, the two shapes of the fused
    push, the two instances of the Gram launch).  A slot refilled before every lane had read it, or a
    barrier phase out of step after a change of ring depth, would show here as a difference."""
    n, M = 296 * 8192 * 2 + 12_345, 10
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 505)
    tokens = [100 + 3 * m for m in range(M)]
    mask, push = (1 << s) - 1, (1 << k) - 1
    ends = []
    for rep in range(2):
        t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
        l_dev = [to_torch_learner(a, "cuda") for a in learners]
        rec_buf = dd.new_records(1)
        for _ in range(20):
            if kind == "push":
                ctx.merge_fragment_push(t_dev, v_dev, l_dev, tokens, mask, 2, ETA, MU, push,
                                        flags=dd.DIAG_STATE, record=rec_buf)
            elif kind == "rda":
                ctx.merge_fragment_rda(t_dev, v_dev, l_dev, tokens, mask, 2, ETA, MU,
                                       flags=dd.DIAG_STATE, record=rec_buf)
            else:
                ctx.merge_fragment(t_dev, v_dev, l_dev, tokens, mask, 2, ETA, MU,
                                   flags=dd.DIAG_STATE, record=rec_buf)
        torch.cuda.synchronize()
        assert dd.read_records(rec_buf)[0].status == 0
        ends.append([t_dev, v_dev, rec_buf.clone()] + [x.view(torch.int16) for x in l_dev])
    assert all(torch.equal(a, b) for a, b in zip(*ends))


@pytest.mark.parametrize("s", [47, 48, 49])
def test_per_learner_norms_around_the_shared_memory_limit(dd, ctx, s):
    """Up to 48 participants the per-participant norms are summed per lane in shared memory and
    reduced once per run of rows; beyond, every piece is reduced at once.  Same result."""
    M = 52
    tokens = [100 + 3 * m for m in range(M)]
    run_case(dd, ctx, 3 * 8192 + 70_001, M, "bf16", tokens, (1 << s) - 1, s, seed=300 + s,
             flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, merges=1)


@pytest.mark.parametrize("shards", [2, 3])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_range_sharded_direct_average_equals_unsharded(dd, ctx, shards, dtype):
    """A fragment cut into contiguous element ranges, as a multi-GPU job holds it (one range per
    rank, no data-path collective): every range is merged by its own call -- here all on one GPU --
    and the ranges' squared norms are added up, which is what the job's one small all-reduce does.
    Result: the oracle's merge of the whole fragment."""
    from paper_2604_21428_b200 import dist as ddist

    n, M = 200_003, 5
    tokens, mask, K = [100, 200, 0, 400, 500], 0b11101, 3
    theta, v, learners = synth.fragment_cpu(n, M, dtype, 4242)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    out_dev = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    o_out = np.zeros(n, dtype=np.uint16)
    ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, ETA, MU, out_bf16=o_out)
    ranges = [ddist.shard_range(n, r, shards) for r in range(shards)]
    assert ranges[0][0] == 0 and ranges[-1][1] == n and all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    recs = [dd.new_records(1) for _ in range(shards)]
    for (lo, hi), rec in zip(ranges, recs):
        ctx.merge_fragment(t_dev[lo:hi], v_dev[lo:hi], [t[lo:hi] for t in l_dev], tokens, mask, K, ETA, MU,
                           n=hi - lo, learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32,
                           flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, out_bf16=out_dev[lo:hi], record=rec)
    torch.cuda.synchronize()
    per_rank = [dd.read_records(rec)[0] for rec in recs]
    # what dist.allreduce_record leaves on every rank: identical participation and weights, summed norms
    total = per_rank[0]
    for r in per_rank[1:]:
        assert (r.status, r.n_part, r.idx, r.w_hat) == (total.status, total.n_part, total.idx, total.w_hat)
    import dataclasses
    total = dataclasses.replace(total, delta_sq=sum(r.delta_sq for r in per_rank),
                                theta_sq=sum(r.theta_sq for r in per_rank), mom_sq=sum(r.mom_sq for r in per_rank),
                                delta_m_sq=[sum(r.delta_m_sq[j] for r in per_rank) for j in range(total.n_part)])
    assert_record_matches(total, ref)
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
    assert floor_rel_err(bf16_bits_to_f32(out_dev), oracle.bf16_to_f32(o_out)) <= TOL_BF16
