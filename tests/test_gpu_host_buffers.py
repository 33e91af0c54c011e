"""Host-buffer entry points for batches and for int4 payloads against the oracle: every operand
sits in (pinned) host memory and streams through the GPU in chunks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import (TOL_BF16, TOL_NORM, TOL_STATE, assert_record_matches, bf16_bits_to_f32,
                         floor_rel_err, to_torch_learner)

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


@pytest.mark.parametrize("dtype,chunk", [("bf16", 0), ("bf16", 4096), ("f32", 8192)])
def test_batched_host_buffers(dd, ctx, dtype, chunk):
    # ragged fragments (one empty, one below a chunk, several chunks with a ragged last one, one below
    # quorum); chunks of successive fragments follow one another through the same staging sets
    rng = np.random.default_rng(17)
    sizes = [30_001, 0, 5, 4096 * 3, 70_003, 9_000]
    M, K = 5, 2
    tokens = rng.integers(1, 1000, size=(len(sizes), M))
    tokens[2, 1] = 0
    masks = [0b11111, 0b00111, 0b10110, 0b01011, 0b11101, 0b00001]      # the last one: below quorum
    hosts, frags = [], []
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, dtype, 300 + p)
        hosts.append((theta, v, learners))
        frags.append(dict(global_=torch.from_numpy(theta.copy()).pin_memory(),
                          momentum=torch.from_numpy(v.copy()).pin_memory(),
                          out_bf16=torch.zeros(n, dtype=torch.bfloat16).pin_memory(),
                          learners=[to_torch_learner(a, "cpu").pin_memory() for a in learners],
                          tokens=[int(t) for t in tokens[p]], quorum_mask=masks[p], K=K, n=n))
    ldt = dd.BF16 if dtype == "bf16" else dd.F32
    for call in range(2):
        recs = ctx.merge_fragments_batched_host(frags, M, ldt, ETA, MU,
                                                flags=dd.DIAG_STATE | dd.DIAG_PER_LEARNER, chunk_elems=chunk)
        for p, (theta, v, learners) in enumerate(hosts):
            n = sizes[p]
            o_out = np.zeros(n, dtype=np.uint16)
            ref = oracle.merge_fragment(theta, v, learners, frags[p]["tokens"], masks[p], K, ETA, MU,
                                        out_bf16=o_out)
            assert_record_matches(recs[p], ref)
            assert floor_rel_err(frags[p]["global_"].numpy(), theta) <= TOL_STATE, (call, p)
            assert floor_rel_err(frags[p]["momentum"].numpy(), v) <= TOL_STATE, (call, p)
            if ref.status == 0 and n:
                assert floor_rel_err(bf16_bits_to_f32(frags[p]["out_bf16"]), oracle.bf16_to_f32(o_out)) <= TOL_BF16
            # both sides start the next call from the oracle's state
            frags[p]["global_"].copy_(torch.from_numpy(theta))
            frags[p]["momentum"].copy_(torch.from_numpy(v))
        assert recs[5].status == dd.STATUS_QUORUM_NOT_MET and recs[1].status == 0
    assert ctx.merge_fragments_batched_host([], M, ldt, ETA, MU) == []


@pytest.mark.parametrize("n,chunk", [(100_003, 0), (100_003, 128 * 40), (127, 0), (5 * 128 * 64, 128 * 64), (0, 0)])
def test_int4_host_buffers(dd, ctx, n, chunk):
    # codes and scales from the ORACLE's quantiser (the learner side), in pinned host memory
    M = 6
    tokens, mask, K = [10, 0, 30, 40, 50, 60], 0b111101, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 88)
    part = [0, 2, 3, 4, 5]
    q = [oracle.quantize_int4(theta, learners[m]) if m in part else None for m in range(M)]
    codes = [None if x is None else x[0] for x in q]
    scales = [None if x is None else x[1] for x in q]
    h_codes = [None if c is None else torch.from_numpy(c.copy()).pin_memory() for c in codes]
    h_scales = [None if s_ is None else torch.from_numpy(s_.copy()).pin_memory() for s_ in scales]
    h_theta = torch.from_numpy(theta.copy()).pin_memory()
    h_v = torch.from_numpy(v.copy()).pin_memory()
    h_out = torch.zeros(n, dtype=torch.bfloat16).pin_memory()
    o_out = np.zeros(n, dtype=np.uint16)
    ref = oracle.merge_fragment_int4(theta, v, codes, scales, tokens, mask, K, ETA, MU, out_bf16=o_out)
    got = ctx.merge_fragment_int4_host(h_theta, h_v, h_codes, h_scales, tokens, mask, K, ETA, MU, n=n,
                                       flags=dd.DIAG_STATE, out_bf16=h_out, chunk_elems=chunk)
    assert (got.status, got.n_part, got.idx) == (ref.status, ref.n_part, ref.idx) and got.n_part == 5
    assert got.w_hat == [float(np.float32(x)) for x in ref.w_hat]
    assert floor_rel_err(h_theta.numpy(), theta) <= TOL_STATE
    assert floor_rel_err(h_v.numpy(), v) <= TOL_STATE
    if n:
        assert floor_rel_err(bf16_bits_to_f32(h_out), oracle.bf16_to_f32(o_out)) <= TOL_BF16
        for name in ("delta_sq", "theta_sq", "mom_sq"):
            a, b = getattr(got, name), getattr(ref, name)
            assert abs(a - b) <= TOL_NORM * abs(b), (name, a, b)
    # a chunk that would split a quantisation block is refused
    with pytest.raises(dd.DDMergeError) as e:
        ctx.merge_fragment_int4_host(h_theta, h_v, h_codes, h_scales, tokens, mask, K, ETA, MU, n=n, chunk_elems=200)
    assert e.value.rc == dd.ERR_INVALID_ARG
    # quorum not met: nothing is transferred or written
    before = h_theta.clone()
    got = ctx.merge_fragment_int4_host(h_theta, h_v, h_codes, h_scales, tokens, mask, 6, ETA, MU, n=n)
    assert got.status == dd.STATUS_QUORUM_NOT_MET and torch.equal(before, h_theta)
