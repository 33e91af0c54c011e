"""The allocation-free batched entry point against the ordinary batched one.

Some users of the library cannot allocate device memory at the time they merge
(their framework owns the GPU's memory, or they may not synchronise the device,
or they run under a no-allocation rule).  For them the library offers
``dd_merge_fragments_batched_noalloc``, whose scratch is a fixed array inside
the library.  This test drives it through the C ABI twice in a row -- the array
keeps the first call's contents, so the second call proves that it is cleared
where it has to be -- and compares every output with the ordinary entry point's.
It lives in a file of its own that is collected last.
"""
import numpy as np
import pytest
import torch

from paper_2604_21428_b200 import synth
from parity_util import TOL_BF16, TOL_NORM, TOL_STATE, floor_rel_err, to_torch_learner

pytestmark = pytest.mark.gpu

ETA, MU = synth.OUTER_LR, synth.OUTER_MU


def _fragments(sizes, M, tokens, masks, K, seed):
    frags = []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", seed + p)
        frags.append(dict(
            global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
            out_bf16=torch.zeros(n, dtype=torch.bfloat16, device="cuda"),
            learners=[to_torch_learner(a, "cuda") for a in learners],
            tokens=[int(t) for t in tokens[p]], quorum_mask=masks[p], K=K, n=n))
    return frags


def test_noalloc_matches_batched_twice_in_a_row():
    from paper_2604_21428_b200 import ddmerge as dd

    torch.cuda.set_device(0)
    rng = np.random.default_rng(99)
    sizes = [3 * 8192 + 11, 70_000, 5, 8192, 123_457]
    M, K = 6, 3
    tokens = rng.integers(1, 1000, size=(len(sizes), M))
    tokens[1, 2] = 0
    masks = [0b111111, 0b101111, 0b000111, 0b000011, 0b110110]     # fragment 3: below quorum
    flags = dd.DIAG_STATE
    a = _fragments(sizes, M, tokens, masks, K, seed=500)            # ordinary entry point
    b = _fragments(sizes, M, tokens, masks, K, seed=500)            # allocation-free entry point
    rec_a, rec_b = dd.new_records(len(sizes)), dd.new_records(len(sizes))
    ctx = dd.Context(0)
    for call in range(2):
        ctx.merge_fragments_batched(a, M, dd.BF16, ETA, MU, flags=flags, records=rec_a)
        dd.merge_fragments_batched_noalloc(b, M, dd.BF16, ETA, MU, flags=flags, records=rec_b)
        torch.cuda.synchronize()
        ra, rb = dd.read_records(rec_a), dd.read_records(rec_b)
        for p in range(len(sizes)):
            assert (rb[p].status, rb[p].n_part, rb[p].idx, rb[p].w_hat) == \
                (ra[p].status, ra[p].n_part, ra[p].idx, ra[p].w_hat), (call, p)
            for name in ("delta_sq", "theta_sq", "mom_sq"):
                x, y = getattr(rb[p], name), getattr(ra[p], name)
                assert abs(x - y) <= TOL_NORM * abs(y), (call, p, name, x, y)
            assert floor_rel_err(b[p]["global_"].cpu().numpy(), a[p]["global_"].cpu().numpy()) <= TOL_STATE
            assert floor_rel_err(b[p]["momentum"].cpu().numpy(), a[p]["momentum"].cpu().numpy()) <= TOL_STATE
            assert floor_rel_err(b[p]["out_bf16"].float().cpu().numpy(),
                                 a[p]["out_bf16"].float().cpu().numpy()) <= TOL_BF16
        assert ra[3].status == dd.STATUS_QUORUM_NOT_MET and ra[0].status == 0
    ctx.close()


def test_noalloc_rejects_what_its_fixed_scratch_cannot_hold():
    from paper_2604_21428_b200 import ddmerge as dd

    torch.cuda.set_device(0)
    M = 2
    one = _fragments([64], M, [[1, 1]], [0b11], 1, seed=7)[0]
    too_many = [one] * (dd.NOALLOC_MAX_FRAGMENTS + 1)
    with pytest.raises(dd.DDMergeError) as e:
        dd.merge_fragments_batched_noalloc(too_many, M, dd.BF16, ETA, MU)
    assert e.value.rc == dd.ERR_TOO_LARGE
    with pytest.raises(dd.DDMergeError) as e:
        dd.merge_fragments_batched_noalloc([one], M, dd.BF16, ETA, MU, flags=dd.DIAG_PER_LEARNER)
    assert e.value.rc == dd.ERR_INVALID_ARG
    torch.cuda.synchronize()
