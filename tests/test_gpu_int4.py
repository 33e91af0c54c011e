"""int4 compression of outer gradients on the GPU: the quantiser's codes and scales are
integer / bit decisions and must equal the oracle's exactly; the merge of compressed
gradients is compared like every other merge."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import TOL_BF16, TOL_NORM, TOL_STATE, bf16_bits_to_f32, floor_rel_err, to_torch_learner

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


def _quantize_gpu(dd, ctx, theta, learner, dtype):
    n = theta.size
    t_dev = torch.from_numpy(theta).cuda()
    l_dev = to_torch_learner(learner, "cuda")
    codes = torch.full(((n + 1) // 2 + 16,), 0xAB, dtype=torch.uint8, device="cuda")     # canary tail
    scales = torch.full(((n + 127) // 128 + 4,), -1.0, dtype=torch.float32, device="cuda")
    ctx.quantize_outer_gradient_int4(t_dev, l_dev, codes, scales, n=n,
                                     learner_dtype=dd.BF16 if dtype == "bf16" else dd.F32)
    torch.cuda.synchronize()
    assert torch.all(codes[(n + 1) // 2:] == 0xAB) and torch.all(scales[(n + 127) // 128:] == -1.0)
    return codes[: (n + 1) // 2], scales[: (n + 127) // 128]


# the largest size spans the four-blocks-at-a-time loop, the one-block loop and a ragged last block
@pytest.mark.parametrize("n", [1, 2, 3, 5, 127, 128, 129, 1000, 8192, 100_003, 4_000_037])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_quantiser_bit_exact(dd, ctx, n, dtype):
    theta, _, learners = synth.fragment_cpu(n, 1, dtype, 900 + n % 13)
    if n >= 256:                                       # one block of exact zeros
        if dtype == "bf16":
            theta[128:256] = oracle.bf16_to_f32(learners[0][128:256])
        else:
            learners[0][128:256] = theta[128:256]
    ref_codes, ref_scales = oracle.quantize_int4(theta, learners[0])
    codes, scales = _quantize_gpu(dd, ctx, theta, learners[0], dtype)
    np.testing.assert_array_equal(scales.cpu().numpy().view(np.uint32), ref_scales.view(np.uint32))
    np.testing.assert_array_equal(codes.cpu().numpy(), ref_codes)


@pytest.mark.parametrize("shift", [0, 1])
def test_quantiser_non_finite_blocks(dd, ctx, shift):
    """Blocks holding NaN or infinite differences: a NaN makes the block's scale NaN, an
    infinity makes it infinite, whichever loop of the kernel handles the block (the unrolled
    one, the one-block one, the unaligned one reached through ``shift``).  NaN scales are
    compared as NaN, everything else bit for bit."""
    nblocks = 4 * 8 * 148 * 8 + 37                      # several rounds of the unrolled loop + a rest
    n = nblocks * 128 - 5
    rng = np.random.default_rng(77)
    theta = np.zeros(n, dtype=np.float32)
    learner = rng.normal(0.0, 1e-3, size=n).astype(np.float32)
    for b in range(0, nblocks, 3):
        lo = b * 128
        kind = (b // 3) % 4
        if kind == 0:
            learner[lo + 5] = np.nan                    # one NaN
        elif kind == 1:
            learner[lo + 4:lo + 8] = np.nan             # a lane's four elements all NaN
        elif kind == 2:
            learner[lo + 9] = np.inf                    # infinity (and finite neighbours)
        else:
            learner[lo + 17] = -np.inf
            learner[lo + 18] = np.nan
    ref_codes, ref_scales = oracle.quantize_int4(theta, learner)
    # device buffers moved off 16-byte alignment by ``shift`` elements
    t_full = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    l_full = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    t_dev, l_dev = t_full[shift:shift + n], l_full[shift:shift + n]
    l_dev.copy_(torch.from_numpy(learner))
    codes = torch.zeros((n + 1) // 2, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(nblocks, dtype=torch.float32, device="cuda")
    ctx.quantize_outer_gradient_int4(t_dev, l_dev, codes, scales, n=n, learner_dtype=dd.F32)
    torch.cuda.synchronize()
    got_s = scales.cpu().numpy()
    assert np.array_equal(np.isnan(got_s), np.isnan(ref_scales)) and np.isnan(ref_scales).sum() > 100
    fin = ~np.isnan(ref_scales)
    np.testing.assert_array_equal(got_s[fin].view(np.uint32), ref_scales[fin].view(np.uint32))
    assert np.isinf(ref_scales).sum() > 100
    np.testing.assert_array_equal(codes.cpu().numpy(), ref_codes)


def test_quantiser_near_ties_and_extreme_scales(dd, ctx):
    """Outer gradients placed on, and one to three ulps beside, the half-integer multiples of
    the block scale -- where rint(d / scale) decides between two codes -- and blocks whose
    scale is tiny, huge or zero.  Codes must still equal the oracle's bit for bit."""
    rng = np.random.default_rng(2024)
    nblocks = 40_000                                    # enough for the four-blocks-at-a-time loop
    n = nblocks * 128
    sc = np.exp(rng.uniform(np.log(1e-6), np.log(1e3), size=nblocks)).astype(np.float32)
    sc[::7] = 1.0                                       # exact ties: d = k + 1/2
    sc[1::97] = np.float32(1e-36)
    sc[2::97] = np.float32(3e33)
    sc[3::97] = np.float32(1e-41)                       # subnormal scale
    k = rng.integers(-7, 7, size=(nblocks, 128)).astype(np.float32)
    ulps = rng.integers(-3, 4, size=(nblocks, 128)).astype(np.float32)
    d = (k + np.float32(0.5)) * sc[:, None]
    d = (d * (np.float32(1.0) + ulps * np.float32(2.0 ** -23))).astype(np.float32)
    d[:, 0] = np.float32(7.0) * sc                      # fixes the block maximum, hence the scale
    d[5::97] = 0.0                                      # all-zero blocks
    learner = (-d).reshape(-1).astype(np.float32)       # Theta = 0: Theta - theta = d exactly
    theta = np.zeros(n, dtype=np.float32)
    ref_codes, ref_scales = oracle.quantize_int4(theta, learner)
    codes, scales = _quantize_gpu(dd, ctx, theta, learner, "f32")
    np.testing.assert_array_equal(scales.cpu().numpy().view(np.uint32), ref_scales.view(np.uint32))
    np.testing.assert_array_equal(codes.cpu().numpy(), ref_codes)
    # the stress is real: both neighbouring codes occur among elements built from the same k
    assert len(np.unique(ref_codes)) > 100


# the largest size gives every thread of the persistent grid more than one 16-element step
@pytest.mark.parametrize("n", [5, 8, 1023, 8192 * 2 + 3, 150_001, 4_000_037])
def test_int4_merge(dd, ctx, n):
    M = 6
    tokens, mask, K = [100, 200, 0, 400, 500, 50], 0b111101, 3
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 950 + n % 7)
    part = [0, 3, 4, 5]                                # mask and tokens > 0 (learner 2 has no tokens)
    q = [oracle.quantize_int4(theta, a) for a in learners]
    codes_d = [torch.from_numpy(q[m][0]).cuda() if m in part else None for m in range(M)]
    scales_d = [torch.from_numpy(q[m][1]).cuda() if m in part else None for m in range(M)]
    codes_h = [q[m][0] if m in part else None for m in range(M)]
    scales_h = [q[m][1] if m in part else None for m in range(M)]
    t_dev, v_dev = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    out_dev = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    rec_buf = dd.new_records(1)
    for k in range(2):
        o_out = np.zeros(n, dtype=np.uint16)
        ref = oracle.merge_fragment_int4(theta, v, codes_h, scales_h, tokens, mask, K, ETA, MU,
                                         out_bf16=o_out)
        ctx.merge_fragment_int4(t_dev, v_dev, codes_d, scales_d, tokens, mask, K, ETA, MU, n=n,
                                flags=dd.DIAG_STATE, out_bf16=out_dev, record=rec_buf)
        torch.cuda.synchronize()
        got = dd.read_records(rec_buf)[0]
        assert (got.status, got.n_part, got.idx) == (ref.status, ref.n_part, ref.idx)
        assert got.w_hat == [float(np.float32(w)) for w in ref.w_hat]
        for name in ("delta_sq", "theta_sq", "mom_sq"):
            a, b = getattr(got, name), getattr(ref, name)
            assert abs(a - b) <= TOL_NORM * abs(b) + 1e-300, (name, a, b)
        assert floor_rel_err(t_dev.cpu().numpy(), theta) <= TOL_STATE
        assert floor_rel_err(v_dev.cpu().numpy(), v) <= TOL_STATE
        assert floor_rel_err(bf16_bits_to_f32(out_dev), oracle.bf16_to_f32(o_out)) <= TOL_BF16
        t_dev.copy_(torch.from_numpy(theta))
        v_dev.copy_(torch.from_numpy(v))
    # quorum not met: nothing written
    before = t_dev.clone()
    ctx.merge_fragment_int4(t_dev, v_dev, codes_d, scales_d, tokens, mask, 5, ETA, MU, n=n,
                            record=rec_buf)
    torch.cuda.synchronize()
    assert dd.read_records(rec_buf)[0].status == dd.STATUS_QUORUM_NOT_MET
    assert torch.equal(before, t_dev)


def test_int4_round_trip_close_to_uncompressed(dd, ctx):
    # quantise on the GPU, merge on the GPU; compare with the uncompressed merge: within half a step
    n, M = 200_000, 8
    theta, v, learners = synth.fragment_cpu(n, M, "bf16", 990)
    t_a, v_a = torch.from_numpy(theta).cuda(), torch.from_numpy(v).cuda()
    t_b, v_b = t_a.clone(), v_a.clone()
    L = [to_torch_learner(a, "cuda") for a in learners]
    codes = [torch.empty((n + 1) // 2, dtype=torch.uint8, device="cuda") for _ in range(M)]
    scales = [torch.empty((n + 127) // 128, dtype=torch.float32, device="cuda") for _ in range(M)]
    for m in range(M):
        ctx.quantize_outer_gradient_int4(t_a, L[m], codes[m], scales[m])
    tokens = [1000 + 37 * m for m in range(M)]
    ctx.merge_fragment_int4(t_a, v_a, codes, scales, tokens, 0xFF, 8, ETA, MU)
    ctx.merge_fragment(t_b, v_b, L, tokens, 0xFF, 8, ETA, MU)
    torch.cuda.synchronize()
    step = max(float(s_.max()) for s_ in scales)
    assert float((v_a - v_b).abs().max()) <= 0.5 * step
    rel = float((v_a - v_b).norm() / v_b.norm())
    assert rel < 0.2                                   # 4 bits: ~10 % noise on one merge's outer gradient
