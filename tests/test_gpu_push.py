"""The merge fused with the push of Theta' into learner copies (Algorithm 2: the syncer sends
the new fragment back; Appendix: alpha = 0 overwrites the learner's copy).  Oracle: its merge,
then its learner-side apply with alpha = 0 on every pushed copy."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import TOL_STATE, floor_rel_err, to_torch_learner

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


def _host(t):
    t = t.cpu()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def _check_pushed(got, want_bits_or_f32, dtype):
    """A pushed copy is Theta' rounded to the learner dtype: equal to the oracle's except where
    the two fp32 states differ by an ulp across a rounding boundary."""
    g = _host(got)
    if dtype == "bf16":
        assert np.mean(g == want_bits_or_f32) > 0.999
        assert floor_rel_err(oracle.bf16_to_f32(g), oracle.bf16_to_f32(want_bits_or_f32)) <= 1e-2
    else:
        assert floor_rel_err(g, want_bits_or_f32) <= TOL_STATE


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("n", [5, 8, 1023, 8192 * 3 + 5, 2 * 296 * 8192 + 8192 + 3])
def test_merge_and_push_single(dd, ctx, n, dtype):
    M = 6
    tokens, mask, K = [100, 200, 0, 400, 500, 50], 0b111101, 3     # participants 0 3 4 5
    push = 0b011110                                                 # pushed 1 2 3 4: two of them not merged
    theta, v, learners = synth.fragment_cpu(n, M, dtype, 600 + n % 11)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    before = [t.clone() for t in l_dev]
    rec = dd.new_records(1)
    ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, ETA, MU)      # theta, v updated in place
    ctx.merge_fragment_push(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU, push, n=n,
                            learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32,
                            flags=dd.DIAG_STATE, record=rec)
    torch.cuda.synchronize()
    got = dd.read_records(rec)[0]
    assert (got.status, got.n_part, got.idx) == (ref.status, ref.n_part, ref.idx) == (0, 4, [0, 3, 4, 5])
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
    for m in range(M):
        if (push >> m) & 1:
            want = learners[m].copy()
            oracle.apply_to_learner(want, theta, 0.0)
            _check_pushed(l_dev[m], want, dtype)
        else:
            assert torch.equal(l_dev[m], before[m]), f"learner {m} was not to be written"
    # quorum not met: nothing merged, nothing pushed
    snap = [t.clone() for t in l_dev]
    t_snap = t_dev.clone()
    ctx.merge_fragment_push(t_dev, v_dev, l_dev, tokens, mask, 5, ETA, MU, push, n=n,
                            learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32, record=rec)
    torch.cuda.synchronize()
    assert dd.read_records(rec)[0].status == dd.STATUS_QUORUM_NOT_MET
    assert torch.equal(t_snap, t_dev) and all(torch.equal(a, b) for a, b in zip(snap, l_dev))


def test_merge_and_push_equals_merge_then_broadcast(dd, ctx):
    # the fused call against the library's own two-call sequence: identical bits
    n, M = 300_011, 8
    tokens = [1000 + 13 * m for m in range(M)]
    mask, K, push = 0b10110111, 4, 0b11111011
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 71)
    a = [torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda(), [to_torch_learner(x, "cuda") for x in learners]]
    b = [torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda(), [to_torch_learner(x, "cuda") for x in learners]]
    ctx.merge_fragment_push(a[0], a[1], a[2], tokens, mask, K, ETA, MU, push)
    ctx.merge_fragment(b[0], b[1], b[2], tokens, mask, K, ETA, MU)
    ctx.broadcast_fragment(b[0], b[2], push, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    for m in range(M):
        assert torch.equal(a[2][m], b[2][m]), m


def test_batched_merge_and_push(dd, ctx):
    sizes = [8192 * 2 + 7, 40_001, 0, 9, 1_500_003]
    M = 4
    rng = np.random.default_rng(12)
    tokens = rng.integers(1, 100, size=(len(sizes), M))
    masks = [0b1111, 0b0111, 0b1111, 0b1010, 0b1101]
    pushes = [0b1111, 0b1000, 0b0001, 0, 0b0110]
    host, frags = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 800 + p)
        host.append((theta, v, learners))
        frags.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                          learners=[to_torch_learner(a, "cuda") for a in learners],
                          tokens=[int(x) for x in tokens[p]], quorum_mask=masks[p], K=2, n=n))
    before = [[t.clone() for t in f["learners"]] for f in frags]
    recs = dd.new_records(len(sizes))
    ctx.merge_fragments_batched_push(frags, pushes, M, dd.BF16, ETA, MU, flags=dd.DIAG_STATE, records=recs)
    torch.cuda.synchronize()
    got = dd.read_records(recs)
    for p, n in enumerate(sizes):
        theta, v, learners = host[p]
        ref = oracle.merge_fragment(theta, v, learners, frags[p]["tokens"], masks[p], 2, ETA, MU)
        assert (got[p].status, got[p].n_part, got[p].idx) == (ref.status, ref.n_part, ref.idx)
        assert floor_rel_err(frags[p]["global_"].cpu().numpy(), theta) <= TOL_STATE
        assert floor_rel_err(frags[p]["momentum"].cpu().numpy(), v) <= TOL_STATE
        for m in range(M):
            if (pushes[p] >> m) & 1 and ref.status == 0 and n:
                want = learners[m].copy()
                oracle.apply_to_learner(want, theta, 0.0)
                _check_pushed(frags[p]["learners"][m], want, "bf16")
            else:
                assert torch.equal(frags[p]["learners"][m], before[p][m])


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_push_to_one_of_many(dd, ctx, dtype):
    # few bytes written per byte read (9 merged, 1 pushed): the launch keeps the ordinary grid and a
    # shallower ring than the write-heavy pushes above; several tiles per CTA and a ragged tail
    n, M = 2 * 296 * 8192 + 4099, 10
    tokens = [50 + 7 * m for m in range(M)]
    mask, K, push = 0b1110111111, 4, 0b0001000000            # learner 6 is pushed to and not merged
    theta, v, learners = synth.fragment_cpu(n, M, dtype, 611)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    before = [t.clone() for t in l_dev]
    rec = dd.new_records(1)
    ref = oracle.merge_fragment(theta, v, learners, tokens, mask, K, ETA, MU)
    ctx.merge_fragment_push(t_dev, v_dev, l_dev, tokens, mask, K, ETA, MU, push, n=n,
                            learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32,
                            flags=dd.DIAG_STATE, record=rec)
    torch.cuda.synchronize()
    got = dd.read_records(rec)[0]
    assert (got.status, got.n_part, got.idx) == (ref.status, ref.n_part, ref.idx) and got.n_part == 9
    assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
    assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
    for m in range(M):
        if (push >> m) & 1:
            want = learners[m].copy()
            oracle.apply_to_learner(want, theta, 0.0)
            _check_pushed(l_dev[m], want, dtype)
        else:
            assert torch.equal(l_dev[m], before[m]), f"learner {m} was not to be written"


def test_batched_push_mixes_pushed_and_plain_fragments(dd, ctx):
    # one launch: fragments with and without a push, above and below 8 participants, about 60 tiles
    # each (CTAs change ring depth between their tiles)
    M = 10
    counts = [9, 4, 10, 8, 2, 9]
    pushes = [0, 0b0000000001, 0b1111111111, 0, 0b0000000110, 0b1000000000]
    sizes = [8192 * 60 + 11 * (p + 1) for p in range(len(counts))]
    rng = np.random.default_rng(41)
    tokens = rng.integers(1, 500, size=(len(sizes), M))
    masks = [(1 << c) - 1 for c in counts]
    host, frags = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 900 + p)
        host.append((theta, v, learners))
        frags.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                          learners=[to_torch_learner(a, "cuda") for a in learners],
                          tokens=[int(x) for x in tokens[p]], quorum_mask=masks[p], K=2, n=n))
    before = [[t.clone() for t in f["learners"]] for f in frags]
    recs = dd.new_records(len(sizes))
    ctx.merge_fragments_batched_push(frags, pushes, M, dd.BF16, ETA, MU, flags=dd.DIAG_STATE, records=recs)
    torch.cuda.synchronize()
    got = dd.read_records(recs)
    for p, n in enumerate(sizes):
        theta, v, learners = host[p]
        ref = oracle.merge_fragment(theta, v, learners, frags[p]["tokens"], masks[p], 2, ETA, MU)
        assert (got[p].status, got[p].n_part, got[p].idx) == (ref.status, ref.n_part, ref.idx)
        assert got[p].n_part == counts[p]
        assert floor_rel_err(frags[p]["global_"].cpu().numpy(), theta) <= TOL_STATE
        assert floor_rel_err(frags[p]["momentum"].cpu().numpy(), v) <= TOL_STATE
        for m in range(M):
            if (pushes[p] >> m) & 1:
                want = learners[m].copy()
                oracle.apply_to_learner(want, theta, 0.0)
                _check_pushed(frags[p]["learners"][m], want, "bf16")
            else:
                assert torch.equal(frags[p]["learners"][m], before[p][m])


def test_push_argument_validation(dd, ctx):
    n, M = 1024, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 5)
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    l_dev = [to_torch_learner(a, "cuda") for a in learners]
    tokens = [1, 1, 1]
    # a pushed learner without a buffer
    with pytest.raises(dd.DDMergeError) as e:
        ctx.merge_fragment_push(t_dev, v_dev, [l_dev[0], l_dev[1], None], tokens, 0b011, 1, ETA, MU, 0b100,
                                n=n, learner_dtype=dd.BF16)
    assert e.value.rc == dd.ERR_INVALID_ARG
    # two pushed learners sharing one buffer
    with pytest.raises(dd.DDMergeError) as e:
        ctx.merge_fragment_push(t_dev, v_dev, [l_dev[0], l_dev[1], l_dev[1]], tokens, 0b001, 1, ETA, MU, 0b110,
                                n=n, learner_dtype=dd.BF16)
    assert e.value.rc == dd.ERR_ALIAS
    # a pushed learner sharing its buffer with a later learner that is only read
    with pytest.raises(dd.DDMergeError) as e:
        ctx.merge_fragment_push(t_dev, v_dev, [l_dev[0], l_dev[1], l_dev[0]], tokens, 0b100, 1, ETA, MU, 0b001,
                                n=n, learner_dtype=dd.BF16)
    assert e.value.rc == dd.ERR_ALIAS
    # bits at or above M are ignored
    ctx.merge_fragment_push(t_dev, v_dev, l_dev, tokens, 0b111, 1, ETA, MU, 0b1000, n=n, learner_dtype=dd.BF16)
    torch.cuda.synchronize()


def test_batched_rda_and_push_equals_rda_then_broadcast(dd, ctx):
    # mixed batch (one plain-average fragment, two radial-directional): the fused push against the
    # library's own merge followed by broadcasts, which the other tests tie to the oracle
    sizes = [30_007, 8192 * 2 + 1, 100_003]
    M = 5
    kinds = [dd.MERGE_AVG, dd.MERGE_RDA, dd.MERGE_RDA]
    masks, pushes = [0b11011, 0b10111, 0b01110], [0b11111, 0b01001, 0b10110]
    tokens = [[5, 9, 2, 7, 3], [4, 4, 8, 1, 6], [2, 3, 5, 7, 11]]

    def make():
        fr = []
        for p, n in enumerate(sizes):
            theta, v, learners = synth.fragment_cpu(n, M, "bf16", 900 + p)
            fr.append(dict(global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
                           learners=[to_torch_learner(a, "cuda") for a in learners], tokens=tokens[p],
                           quorum_mask=masks[p], K=2, n=n))
        return fr

    a, b = make(), make()
    ctx.merge_fragments_batched_rda(a, M, dd.BF16, ETA, MU, merge_kinds=kinds, push_masks=pushes)
    ctx.merge_fragments_batched_rda(b, M, dd.BF16, ETA, MU, merge_kinds=kinds)
    for p in range(len(sizes)):
        ctx.broadcast_fragment(b[p]["global_"], b[p]["learners"], pushes[p], 0.0)
    torch.cuda.synchronize()
    for p in range(len(sizes)):
        assert torch.equal(a[p]["global_"], b[p]["global_"]) and torch.equal(a[p]["momentum"], b[p]["momentum"])
        for m in range(M):
            assert torch.equal(a[p]["learners"][m], b[p]["learners"][m]), (p, m)
