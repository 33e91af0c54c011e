"""Parity at full workload sizes, in the launch configuration bench.py times.

The oracle cannot run 5e8 x 24 elements in a test, so the CUDA result is checked
(a) element by element on sampled windows whose inputs were copied out BEFORE the
merge and fed to the oracle, and (b) through properties that hold at any size:
participation and weights (data independent), and the squared norms against
float64 reductions done with torch on the device.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import TOL_NORM, TOL_STATE, floor_rel_err

pytestmark = pytest.mark.gpu

ETA, MU = synth.OUTER_LR, synth.OUTER_MU
WINDOW = 1 << 16


def _free_bytes():
    """Free device memory once this process has returned what earlier tests left cached."""
    import gc

    gc.collect()
    torch.cuda.empty_cache()
    return torch.cuda.mem_get_info()[0]


def _windows(n, count, rng):
    """First, last and `count` random windows (8-element aligned starts)."""
    if n <= 2 * WINDOW:
        return [(0, n)]
    starts = {0, n - WINDOW - (n - WINDOW) % 8}
    while len(starts) < count + 2:
        starts.add(int(rng.integers(0, (n - WINDOW) // 8)) * 8)
    return [(s, s + WINDOW) for s in sorted(starts)]


def _to_host_learner(t):
    t = t.cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def _expected_delta_sq(theta, learners, idx, w_hat, chunk=1 << 24):
    """||sum_j w_j (Theta - theta_j)||^2 in float64 with torch, chunk by chunk."""
    total = 0.0
    n = theta.numel()
    w = [float(x) for x in w_hat]
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        T = theta[lo:hi].double()
        d = torch.zeros_like(T)
        for j, m in enumerate(idx):
            d += w[j] * (T - learners[m][lo:hi].double())
        total += float((d * d).sum())
    return total


def _sq(t, chunk=1 << 26):
    return sum(float((t[lo:lo + chunk].double() ** 2).sum()) for lo in range(0, t.numel(), chunk))


def _run(name, n_windows, merges):
    from paper_2604_21428_b200 import ddmerge as dd

    w = synth.workload(name)
    # resident: the participants' copies, Theta and v (the algorithmic bytes count Theta and v twice)
    b_theta = 2 if w.learner_dtype == "bf16" else 4
    need = sum(n * (8 + b_theta * sum(1 for m in range(w.M) if (w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0))
               for p, n in enumerate(w.fragment_sizes))
    free = _free_bytes()
    if free < need + (4 << 30):
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    dev = torch.device("cuda", 0)
    ldt = torch.bfloat16 if w.learner_dtype == "bf16" else torch.float32
    ldtype = dd.BF16 if w.learner_dtype == "bf16" else dd.F32
    rng = np.random.default_rng(1234)
    frags = []
    for p, n in enumerate(w.fragment_sizes):
        part = [m for m in range(w.M) if (w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0]
        theta = torch.empty(n, dtype=torch.float32, device=dev)
        mom = torch.empty(n, dtype=torch.float32, device=dev)
        learners = [torch.empty(n, dtype=ldt, device=dev) if m in part else None for m in range(w.M)]
        synth.fill_fragment_gpu(theta, mom, learners, seed=w.seed * 1000 + p)
        frags.append(dict(global_=theta, momentum=mom, learners=learners, part=part,
                          tokens=[int(x) for x in w.tokens[p]], quorum_mask=w.masks[p], K=w.K, n=n,
                          windows=_windows(n, n_windows, rng)))
    ctx = dd.Context(0)
    records = dd.new_records(w.P, device=dev)
    flags = dd.DIAG_STATE
    for k in range(merges):
        # copy the sampled inputs out before the merge overwrites the state
        saved = []
        for f in frags:
            per = []
            for lo, hi in f["windows"]:
                per.append((f["global_"][lo:hi].cpu().numpy().copy(),
                            f["momentum"][lo:hi].cpu().numpy().copy(),
                            [None if t is None else _to_host_learner(t[lo:hi]) for t in f["learners"]]))
            saved.append(per)
        st, idx0 = oracle.participants(frags[0]["quorum_mask"], frags[0]["tokens"], frags[0]["K"])
        expect_dsq = None
        if k == 0:
            _, w0, _ = oracle.weights(frags[0]["tokens"], None, idx0)
            expect_dsq = _expected_delta_sq(frags[0]["global_"], frags[0]["learners"], idx0,
                                            [np.float32(x) for x in w0])
        if w.P == 1:
            f = frags[0]
            ctx.merge_fragment(f["global_"], f["momentum"], f["learners"], f["tokens"],
                               f["quorum_mask"], f["K"], ETA, MU, n=f["n"], learner_dtype=ldtype,
                               flags=flags, record=records)
        else:
            ctx.merge_fragments_batched(frags, w.M, ldtype, ETA, MU, flags=flags, records=records)
        torch.cuda.synchronize()
        recs = dd.read_records(records)
        for p, f in enumerate(frags):
            rec = recs[p]
            for (lo, hi), (t0, v0, ls) in zip(f["windows"], saved[p]):
                ref = oracle.merge_fragment(t0, v0, ls, f["tokens"], f["quorum_mask"], f["K"], ETA, MU)
                assert (rec.status, rec.n_part, rec.idx) == (ref.status, ref.n_part, ref.idx)
                assert rec.w_hat == [float(np.float32(x)) for x in ref.w_hat]
                e_t = floor_rel_err(f["global_"][lo:hi].cpu().numpy(), t0)
                e_v = floor_rel_err(f["momentum"][lo:hi].cpu().numpy(), v0)
                assert e_t <= TOL_STATE and e_v <= TOL_STATE, (k, p, lo, e_t, e_v)
            assert rec.n_part == len(f["part"])
            assert abs(rec.theta_sq - _sq(f["global_"])) <= TOL_NORM * rec.theta_sq
            assert abs(rec.mom_sq - _sq(f["momentum"])) <= TOL_NORM * rec.mom_sq
        if expect_dsq is not None:
            assert abs(recs[0].delta_sq - expect_dsq) <= TOL_NORM * expect_dsq, (recs[0].delta_sq, expect_dsq)
    ctx.close()


def test_scale500m_full_size_sampled():
    _run("scale500m", n_windows=10, merges=2)


def test_dense150m_full_size_batched_sampled():
    _run("dense150m", n_windows=4, merges=2)


def test_dense1b3_full_size_batched_sampled():
    _run("dense1b3", n_windows=2, merges=1)


def test_moe4b_full_size_batched_sampled():
    _run("moe4b", n_windows=1, merges=1)


def test_scale500m_full_size_int4_sampled():
    """The compressed merge at the size and participant count bench.py --merge int4 times:
    every participant's copy is generated, quantised on the GPU and dropped; the oracle
    quantises and merges the sampled windows (block aligned) from the saved inputs."""
    from paper_2604_21428_b200 import ddmerge as dd

    w = synth.workload("scale500m")
    n = w.fragment_sizes[0]
    free = _free_bytes()
    if free < (24 << 30):
        pytest.skip("needs 24 GiB of device memory")
    dev = torch.device("cuda", 0)
    tokens = [int(x) for x in w.tokens[0]]
    mask, K = w.masks[0], w.K
    part = [m for m in range(w.M) if (mask >> m) & 1 and tokens[m] > 0]
    rng = np.random.default_rng(4321)
    windows = [(lo - lo % 128, lo - lo % 128 + WINDOW) for lo, _ in _windows(n, 4, rng)]
    g = torch.Generator(device=dev).manual_seed(77)
    theta = torch.randn(n, generator=g, device=dev) * synth.THETA_STD
    mom = torch.randn(n, generator=g, device=dev) * 1e-3
    ctx = dd.Context(0)
    codes, scales, saved_l = [None] * w.M, [None] * w.M, [None] * w.M
    for m in part:
        learner = (theta + torch.randn(n, generator=g, device=dev) * synth.LEARNER_NOISE_STD).to(torch.bfloat16)
        codes[m] = torch.empty((n + 1) // 2, dtype=torch.uint8, device=dev)
        scales[m] = torch.empty((n + 127) // 128, dtype=torch.float32, device=dev)
        ctx.quantize_outer_gradient_int4(theta, learner, codes[m], scales[m])
        saved_l[m] = [_to_host_learner(learner[lo:hi]) for lo, hi in windows]
        del learner
    saved = [(theta[lo:hi].cpu().numpy().copy(), mom[lo:hi].cpu().numpy().copy()) for lo, hi in windows]
    records = dd.new_records(1, device=dev)
    ctx.merge_fragment_int4(theta, mom, codes, scales, tokens, mask, K, ETA, MU, n=n,
                            flags=dd.DIAG_STATE, record=records)
    torch.cuda.synchronize()
    rec = dd.read_records(records)[0]
    for k, (lo, hi) in enumerate(windows):
        t0, v0 = saved[k]
        q = [oracle.quantize_int4(t0, saved_l[m][k]) if m in part else None for m in range(w.M)]
        # the quantiser is bit-exact: codes and scales of the window as the GPU wrote them
        for m in part:
            np.testing.assert_array_equal(codes[m][lo // 2:hi // 2].cpu().numpy(), q[m][0])
            np.testing.assert_array_equal(scales[m][lo // 128:hi // 128].cpu().numpy().view(np.uint32),
                                          q[m][1].view(np.uint32))
        ref = oracle.merge_fragment_int4(t0, v0, [None if x is None else x[0] for x in q],
                                         [None if x is None else x[1] for x in q], tokens, mask, K, ETA, MU)
        assert (rec.status, rec.n_part, rec.idx) == (ref.status, ref.n_part, ref.idx)
        assert rec.w_hat == [float(np.float32(x)) for x in ref.w_hat]
        assert floor_rel_err(theta[lo:hi].cpu().numpy(), t0) <= TOL_STATE
        assert floor_rel_err(mom[lo:hi].cpu().numpy(), v0) <= TOL_STATE
    assert abs(rec.theta_sq - _sq(theta)) <= TOL_NORM * rec.theta_sq
    assert abs(rec.mom_sq - _sq(mom)) <= TOL_NORM * rec.mom_sq
    ctx.close()


def test_scale500m_full_size_rda_properties():
    """The radial-directional merge at bench size.  Its result depends on whole-fragment norms,
    so the oracle cannot take a window; what is checked holds at any size: per-participant
    norms against float64 device reductions, ||Delta|| = sum_m w_m ||Delta_m|| (the defining
    property of the merge), and on sampled windows v' - mu v = Delta = c u, u the weighted mean
    of unit directions and c the factor that whole-fragment float64 reductions fix."""
    from paper_2604_21428_b200 import ddmerge as dd

    w = synth.workload("scale500m")
    n = w.fragment_sizes[0]
    free = _free_bytes()
    if free < (36 << 30):
        pytest.skip("needs 36 GiB of device memory")
    dev = torch.device("cuda", 0)
    tokens = [int(x) for x in w.tokens[0]]
    mask, K = w.masks[0], w.K
    part = [m for m in range(w.M) if (mask >> m) & 1 and tokens[m] > 0]
    theta = torch.empty(n, dtype=torch.float32, device=dev)
    mom = torch.empty(n, dtype=torch.float32, device=dev)
    learners = [torch.empty(n, dtype=torch.bfloat16, device=dev) if m in part else None for m in range(w.M)]
    synth.fill_fragment_gpu(theta, mom, learners, seed=99)
    mom.normal_(0.0, 1e-3, generator=torch.Generator(device=dev).manual_seed(5))
    chunk = 1 << 25
    norms = []
    for m in part:
        acc = 0.0
        for lo in range(0, n, chunk):
            d = theta[lo:lo + chunk].double() - learners[m][lo:lo + chunk].double()
            acc += float((d * d).sum())
        norms.append(acc ** 0.5)
    st, idx = oracle.participants(mask, tokens, K)
    _, w_hat, _ = oracle.weights(tokens, None, idx)
    wf = [float(np.float32(x)) for x in w_hat]
    u_sq = 0.0                                           # ||sum_j w_j Delta_j / ||Delta_j|| ||^2
    for lo in range(0, n, chunk):
        T = theta[lo:lo + chunk].double()
        u = torch.zeros_like(T)
        for j, m in enumerate(part):
            u += (wf[j] / norms[j]) * (T - learners[m][lo:lo + chunk].double())
        u_sq += float((u * u).sum())
    radial = sum(wf[j] * norms[j] for j in range(len(part)))
    c_expected = radial / u_sq ** 0.5
    rng = np.random.default_rng(99)
    windows = _windows(n, 3, rng)
    saved = [(theta[lo:hi].double().cpu().numpy(), mom[lo:hi].double().cpu().numpy(),
              [learners[m][lo:hi].double().cpu().numpy() for m in part]) for lo, hi in windows]
    ctx = dd.Context(0)
    records = dd.new_records(1, device=dev)
    ctx.merge_fragment_rda(theta, mom, learners, tokens, mask, K, ETA, MU, n=n, learner_dtype=dd.BF16,
                           flags=dd.DIAG_STATE, record=records)
    torch.cuda.synchronize()
    rec = dd.read_records(records)[0]
    assert (rec.status, rec.n_part, rec.idx) == (st, len(idx), list(idx))
    assert rec.w_hat == wf
    for j in range(len(part)):
        assert abs(rec.delta_m_sq[j] - norms[j] ** 2) <= TOL_NORM * norms[j] ** 2
    assert abs(rec.delta_sq ** 0.5 - radial) <= 1e-5 * radial
    for (lo, hi), (t0, v0, ls) in zip(windows, saved):
        u = sum(wf[j] / norms[j] * (t0 - ls[j]) for j in range(len(part)))
        delta = mom[lo:hi].double().cpu().numpy() - MU * v0           # v' = mu v + Delta
        # Delta = c u with one factor for the whole fragment, fixed by the norms
        assert floor_rel_err(delta, c_expected * u) <= TOL_STATE
    assert abs(rec.theta_sq - _sq(theta)) <= TOL_NORM * rec.theta_sq
    assert abs(rec.mom_sq - _sq(mom)) <= TOL_NORM * rec.mom_sq
    ctx.close()


def test_fragment_beyond_32_bit_offsets():
    """One fragment of 2^32 + 24,581 elements (17 GB of Theta, 17 GB of v, one participating bf16
    copy, merged and pushed to): element indices pass 2^32 and byte offsets pass 2^32, 2^33 and
    2^34.  Windows sit on each of those boundaries; the oracle merges them from inputs saved
    before the launch."""
    from paper_2604_21428_b200 import ddmerge as dd

    n = (1 << 32) + 3 * 8192 + 5
    free = _free_bytes()
    if free < 10 * n + (6 << 30):
        pytest.skip("needs 46 GiB of device memory")
    dev = torch.device("cuda", 0)
    theta = torch.empty(n, dtype=torch.float32, device=dev)
    mom = torch.empty(n, dtype=torch.float32, device=dev)
    copy = torch.empty(n, dtype=torch.bfloat16, device=dev)
    synth.fill_fragment_gpu(theta, mom, [copy], seed=4242)
    learners = [None, copy]                              # learner 0 is absent: null pointer
    tokens, mask, K = [0, 12345], 0b10, 1
    half = WINDOW // 2
    centres = [half, 1 << 29, 1 << 30, 1 << 31, (1 << 32) - 8192, 1 << 32, n - half]
    starts = [max(0, min(n - WINDOW, c - half)) for c in centres]
    windows = [(lo, lo + WINDOW) for lo in starts]
    saved = [(theta[lo:hi].cpu().numpy().copy(), mom[lo:hi].cpu().numpy().copy(),
              [None, _to_host_learner(copy[lo:hi])]) for lo, hi in windows]
    ctx = dd.Context(0)
    records = dd.new_records(1, device=dev)
    # merged and pushed in one launch: the copy is overwritten with Theta' (bf16) in place
    ctx.merge_fragment_push(theta, mom, learners, tokens, mask, K, ETA, MU, 0b10, n=n,
                            learner_dtype=dd.BF16, flags=dd.DIAG_STATE, record=records)
    torch.cuda.synchronize()
    rec = dd.read_records(records)[0]
    assert (rec.status, rec.n_part, rec.idx[:1]) == (0, 1, [1])
    for (lo, hi), (t0, v0, ls) in zip(windows, saved):
        oracle.merge_fragment(t0, v0, ls, tokens, mask, K, ETA, MU)
        e_t = floor_rel_err(theta[lo:hi].cpu().numpy(), t0)
        e_v = floor_rel_err(mom[lo:hi].cpu().numpy(), v0)
        assert e_t <= TOL_STATE and e_v <= TOL_STATE, (lo, e_t, e_v)
        oracle.apply_to_learner(ls[1], t0, 0.0)
        assert np.mean(_to_host_learner(copy[lo:hi]) == ls[1]) > 0.999, lo
    assert abs(rec.theta_sq - _sq(theta)) <= TOL_NORM * rec.theta_sq
    assert abs(rec.mom_sq - _sq(mom)) <= TOL_NORM * rec.mom_sq
    ctx.close()


def test_int4_fragment_beyond_32_bit_offsets():
    """The quantiser and the compressed merge on 2^32 + 12,421 elements: windows on the element
    index 2^32 and on the byte-offset boundaries of Theta / v (2^32 ... 2^34) and of the codes."""
    from paper_2604_21428_b200 import ddmerge as dd

    n = (1 << 32) + 97 * 128 + 5
    free = _free_bytes()
    if free < 11 * n + (6 << 30):
        pytest.skip("needs 50 GiB of device memory")
    dev = torch.device("cuda", 0)
    theta = torch.empty(n, dtype=torch.float32, device=dev)
    mom = torch.empty(n, dtype=torch.float32, device=dev)
    copy = torch.empty(n, dtype=torch.bfloat16, device=dev)
    synth.fill_fragment_gpu(theta, mom, [copy], seed=777)
    codes = torch.empty((n + 1) // 2, dtype=torch.uint8, device=dev)
    scales = torch.empty((n + 127) // 128, dtype=torch.float32, device=dev)
    ctx = dd.Context(0)
    ctx.quantize_outer_gradient_int4(theta, copy, codes, scales)
    half = WINDOW // 2
    centres = [half, 1 << 30, 1 << 31, 1 << 32, n]
    starts = [max(0, min(n - WINDOW, c - half)) // 128 * 128 for c in centres]
    windows = [(lo, min(n, lo + WINDOW + 128)) for lo in starts]      # the last one ends on the ragged block
    saved = [(theta[lo:hi].cpu().numpy().copy(), mom[lo:hi].cpu().numpy().copy(),
              _to_host_learner(copy[lo:hi])) for lo, hi in windows]
    del copy
    tokens, mask, K = [777], 0b1, 1
    records = dd.new_records(1, device=dev)
    ctx.merge_fragment_int4(theta, mom, [codes], [scales], tokens, mask, K, ETA, MU, n=n,
                            flags=dd.DIAG_STATE, record=records)
    torch.cuda.synchronize()
    rec = dd.read_records(records)[0]
    assert (rec.status, rec.n_part) == (0, 1)
    for (lo, hi), (t0, v0, l0) in zip(windows, saved):
        q_codes, q_scales = oracle.quantize_int4(t0, l0)
        np.testing.assert_array_equal(codes[lo // 2:(hi + 1) // 2].cpu().numpy(), q_codes)
        np.testing.assert_array_equal(scales[lo // 128:(hi + 127) // 128].cpu().numpy().view(np.uint32),
                                      q_scales.view(np.uint32))
        oracle.merge_fragment_int4(t0, v0, [q_codes], [q_scales], tokens, mask, K, ETA, MU)
        assert floor_rel_err(theta[lo:hi].cpu().numpy(), t0) <= TOL_STATE, lo
        assert floor_rel_err(mom[lo:hi].cpu().numpy(), v0) <= TOL_STATE, lo
    assert abs(rec.theta_sq - _sq(theta)) <= TOL_NORM * rec.theta_sq
    ctx.close()
