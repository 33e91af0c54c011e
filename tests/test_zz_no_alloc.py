"""The allocation-free batched entry point against the ordinary batched one and the oracle.

Some users of the library cannot allocate device memory at the time they merge
(their framework owns the GPU's memory, or they may not synchronise the device,
or they run under a no-allocation rule).  For them the library offers
``dd_merge_fragments_batched_noalloc``, whose scratch is a fixed array inside
the library.  These tests drive it through the C ABI twice in a row -- the array
keeps the first call's contents, so the second call proves that it is cleared
where it has to be -- and compare every output with the ordinary entry point's;
the first call, which starts from the seeded inputs, is also compared element by
element with the CPU oracle.  The file is collected last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import (TOL_BF16, TOL_NORM, TOL_STATE, assert_record_matches, bf16_bits_to_f32,
                         floor_rel_err, to_torch_learner)

pytestmark = pytest.mark.gpu

ETA, MU = synth.OUTER_LR, synth.OUTER_MU


def _fragments(sizes, M, tokens, masks, K, seed, dtype="bf16"):
    """Device fragments and the host arrays they were made from."""
    frags, hosts = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, dtype, seed + p)
        hosts.append((theta, v, learners))
        frags.append(dict(
            global_=torch.from_numpy(theta).cuda(), momentum=torch.from_numpy(v).cuda(),
            out_bf16=torch.zeros(n, dtype=torch.bfloat16, device="cuda"),
            learners=[to_torch_learner(a, "cuda") for a in learners],
            tokens=[int(t) for t in tokens[p]], quorum_mask=masks[p], K=K, n=n))
    return frags, hosts


def _compare_with_batched(dd, a, b, rec_a, rec_b, where):
    ra, rb = dd.read_records(rec_a), dd.read_records(rec_b)
    for p in range(len(a)):
        assert (rb[p].status, rb[p].n_part, rb[p].idx, rb[p].w_hat) == \
            (ra[p].status, ra[p].n_part, ra[p].idx, ra[p].w_hat), (where, p)
        for name in ("delta_sq", "theta_sq", "mom_sq"):
            x, y = getattr(rb[p], name), getattr(ra[p], name)
            assert abs(x - y) <= TOL_NORM * abs(y), (where, p, name, x, y)
        assert floor_rel_err(b[p]["global_"].cpu().numpy(), a[p]["global_"].cpu().numpy()) <= TOL_STATE
        assert floor_rel_err(b[p]["momentum"].cpu().numpy(), a[p]["momentum"].cpu().numpy()) <= TOL_STATE
        assert floor_rel_err(b[p]["out_bf16"].float().cpu().numpy(),
                             a[p]["out_bf16"].float().cpu().numpy()) <= TOL_BF16
    return ra


def _compare_with_oracle(dd, b, hosts, rec_b, K):
    """First call only: the device state still equals the seeded host arrays, which the oracle
    then updates in place."""
    for p, (rec, f, (theta, v, learners)) in enumerate(zip(dd.read_records(rec_b), b, hosts)):
        n = f["n"]
        out = np.zeros(n, dtype=np.uint16)
        ref = oracle.merge_fragment(theta, v, learners, f["tokens"], f["quorum_mask"], K, ETA, MU,
                                    out_bf16=out)
        assert_record_matches(rec, ref, per_learner=False)
        assert floor_rel_err(f["global_"].cpu().numpy(), theta) <= TOL_STATE, p
        assert floor_rel_err(f["momentum"].cpu().numpy(), v) <= TOL_STATE, p
        if ref.status == 0 and n:
            got = bf16_bits_to_f32(f["out_bf16"])
            assert floor_rel_err(got, oracle.bf16_to_f32(out)) <= TOL_BF16, p


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
    a, _ = _fragments(sizes, M, tokens, masks, K, seed=500)         # ordinary entry point
    b, hosts = _fragments(sizes, M, tokens, masks, K, seed=500)     # allocation-free entry point
    rec_a, rec_b = dd.new_records(len(sizes)), dd.new_records(len(sizes))
    ctx = dd.Context(0)
    for call in range(2):
        ctx.merge_fragments_batched(a, M, dd.BF16, ETA, MU, flags=flags, records=rec_a)
        dd.merge_fragments_batched_noalloc(b, M, dd.BF16, ETA, MU, flags=flags, records=rec_b)
        torch.cuda.synchronize()
        ra = _compare_with_batched(dd, a, b, rec_a, rec_b, call)
        assert ra[3].status == dd.STATUS_QUORUM_NOT_MET and ra[0].status == 0
        if call == 0:
            _compare_with_oracle(dd, b, hosts, rec_b, K)
    ctx.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_noalloc_largest_batch_both_dtypes(dtype):
    """Exactly DD_NOALLOC_MAX_FRAGMENTS fragments -- the most the fixed scratch holds -- with
    ragged sizes (an empty fragment, fewer than eight elements, whole tiles, ragged ends) and
    more tiles than the grid has CTAs, for float32 and bf16 learner copies.  Two calls in a row
    against the ordinary entry point, the first also against the oracle; the second call must
    leave the amount of free device memory exactly as it found it."""
    from paper_2604_21428_b200 import ddmerge as dd

    torch.cuda.set_device(0)
    ctx = dd.Context(0)
    ldt = dd.F32 if dtype == "f32" else dd.BF16
    grid, _, tile = ctx.launch_geometry(ldt)
    P, M, K = dd.NOALLOC_MAX_FRAGMENTS, 3, 2
    rng = np.random.default_rng(2718)
    sizes = [0, 5, 7, 8, 9, tile, tile + 1, 3 * tile - 3] + \
            [int(x) for x in rng.integers(1, 4 * tile, size=P - 11)] + \
            [120 * tile + 13, 130 * tile, 77 * tile + 4]
    assert len(sizes) == P and sum((n + tile - 1) // tile for n in sizes) > grid
    tokens = rng.integers(1, 10_000, size=(P, M))
    masks = [int(x) for x in rng.integers(3, 8, size=P)]            # one to three learners: some fragments fall below the quorum
    masks[4] = 0b001                                                # one fragment below quorum
    flags = dd.DIAG_STATE
    a, _ = _fragments(sizes, M, tokens, masks, K, seed=900, dtype=dtype)
    b, hosts = _fragments(sizes, M, tokens, masks, K, seed=900, dtype=dtype)
    rec_a, rec_b = dd.new_records(P), dd.new_records(P)
    for call in range(2):
        ctx.merge_fragments_batched(a, M, ldt, ETA, MU, flags=flags, records=rec_a)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        dd.merge_fragments_batched_noalloc(b, M, ldt, ETA, MU, flags=flags, records=rec_b)
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed free device memory"
        ra = _compare_with_batched(dd, a, b, rec_a, rec_b, call)
        assert ra[4].status == dd.STATUS_QUORUM_NOT_MET
        if call == 0:
            _compare_with_oracle(dd, b, hosts, rec_b, K)
    ctx.close()


def test_noalloc_rejects_what_its_fixed_scratch_cannot_hold():
    from paper_2604_21428_b200 import ddmerge as dd

    torch.cuda.set_device(0)
    M = 2
    one = _fragments([64], M, [[1, 1]], [0b11], 1, seed=7)[0][0]
    too_many = [one] * (dd.NOALLOC_MAX_FRAGMENTS + 1)
    with pytest.raises(dd.DDMergeError) as e:
        dd.merge_fragments_batched_noalloc(too_many, M, dd.BF16, ETA, MU)
    assert e.value.rc == dd.ERR_TOO_LARGE
    with pytest.raises(dd.DDMergeError) as e:
        dd.merge_fragments_batched_noalloc([one], M, dd.BF16, ETA, MU, flags=dd.DIAG_PER_LEARNER)
    assert e.value.rc == dd.ERR_INVALID_ARG
    torch.cuda.synchronize()
