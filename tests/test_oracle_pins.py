"""Pins for the CPU oracle: what the paper and the mathematics fix.

Each test checks the oracle against something that is not the oracle: a closed
form, a special case that reduces to a plain mean, a brute-force enumeration, or
an independent library routine (torch.optim.SGD, torch's bf16 cast).
"""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth


def _frag(n=4096, M=4, dtype="f32", seed=0):
    return synth.fragment_cpu(n, M, dtype, seed)


def _as_f64(learner):
    if learner.dtype == np.uint16:
        return oracle.bf16_to_f32(learner).astype(np.float64)
    return learner.astype(np.float64)


def _full_mask(M):
    return (1 << M) - 1


# ---- Eq. 2: equal tokens, everyone in quorum -> plain mean -----------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_equal_tokens_is_plain_average(dtype):
    theta, v, learners = _frag(M=5, dtype=dtype, seed=11)
    theta0 = theta.astype(np.float64)
    mean = np.mean([_as_f64(a) for a in learners], axis=0)
    rec = oracle.merge_fragment(theta, v, learners, [777] * 5, _full_mask(5), 5, 1.0, 0.0)
    assert rec.status == 0 and rec.idx == [0, 1, 2, 3, 4]
    np.testing.assert_allclose(rec.w_hat, [0.2] * 5, rtol=1e-15)
    # mu = 0: v' = Delta = Theta - mean(theta_m); lr 1: Theta' = mean(theta_m)
    np.testing.assert_allclose(v, (theta0 - mean).astype(np.float32), rtol=0, atol=1e-9)
    np.testing.assert_allclose(theta, mean.astype(np.float32), rtol=1e-6, atol=1e-9)


# ---- Section 2: averaging == SGD with lr 1 (token-weighted) -----------------------

def test_lr1_mu0_is_token_weighted_mean():
    theta, v, learners = _frag(M=4, seed=5)
    tokens = [1000, 3000, 500, 2500]
    w = np.array(tokens, dtype=np.float64) / sum(tokens)
    expect = sum(w[m] * _as_f64(learners[m]) for m in range(4))
    oracle.merge_fragment(theta, v, learners, tokens, _full_mask(4), 1, 1.0, 0.0)
    np.testing.assert_allclose(theta, expect, rtol=2e-6, atol=1e-9)


def test_sign_is_global_minus_learner():
    # One learner strictly above the global everywhere: Delta < 0 and Theta moves up.
    n = 64
    theta = np.full(n, 1.0, dtype=np.float32)
    v = np.zeros(n, dtype=np.float32)
    learners = [np.full(n, 1.5, dtype=np.float32)]
    oracle.merge_fragment(theta, v, learners, [10], 1, 1, 0.5, 0.0)
    np.testing.assert_array_equal(v, np.full(n, -0.5, dtype=np.float32))
    np.testing.assert_array_equal(theta, np.full(n, 1.25, dtype=np.float32))


# ---- Section 4: absent learner == weight 0 ----------------------------------------

def test_masked_or_zero_token_learner_has_no_effect():
    theta, v, learners = _frag(M=4, seed=7)
    tokens = [100, 200, 300, 400]
    t_ref, v_ref = theta.copy(), v.copy()
    ref = oracle.merge_fragment(t_ref, v_ref, [learners[0], learners[2]], [100, 300], 0b11, 2,
                                0.7, 0.9)
    # (a) learner 1 masked out and filled with NaN, learner 3 reports zero tokens + Inf data
    poisoned = [learners[0], np.full_like(learners[1], np.nan), learners[2],
                np.full_like(learners[3], np.inf)]
    t_a, v_a = theta.copy(), v.copy()
    rec = oracle.merge_fragment(t_a, v_a, poisoned, [100, 200, 300, 0], 0b1101, 2, 0.7, 0.9)
    assert rec.idx == [0, 2] and rec.n_part == 2
    np.testing.assert_array_equal(t_a, t_ref)
    np.testing.assert_array_equal(v_a, v_ref)
    assert rec.w_hat == ref.w_hat and rec.delta_sq == ref.delta_sq
    # (b) the same with null pointers for the absent learners
    t_b, v_b = theta.copy(), v.copy()
    oracle.merge_fragment(t_b, v_b, [learners[0], None, learners[2], None], tokens, 0b0101, 2,
                          0.7, 0.9)
    np.testing.assert_array_equal(t_b, t_ref)
    np.testing.assert_array_equal(v_b, v_ref)


def test_quorum_not_met_leaves_state_untouched():
    theta, v, learners = _frag(M=3, seed=2)
    v[:] = 0.25
    t0, v0 = theta.copy(), v.copy()
    rec = oracle.merge_fragment(theta, v, learners, [5, 0, 7], 0b111, 3, 0.7, 0.9)
    assert rec.status == oracle.STATUS_QUORUM_NOT_MET and rec.n_part == 2
    np.testing.assert_array_equal(theta, t0)
    np.testing.assert_array_equal(v, v0)
    # K = 0 behaves as K = 1: an empty set never proceeds
    rec = oracle.merge_fragment(theta, v, learners, [0, 0, 0], 0b111, 0, 0.7, 0.9)
    assert rec.status == oracle.STATUS_QUORUM_NOT_MET and rec.n_part == 0


# ---- symmetry of the weighted sum -------------------------------------------------

def test_permutation_invariance():
    M = 6
    theta, v, learners = _frag(M=M, dtype="bf16", seed=3)
    v[:] = np.random.default_rng(0).normal(0, 1e-3, v.shape).astype(np.float32)
    tokens = [11, 0, 500, 42, 7, 1000]
    mask = 0b111011
    steps = [1, 1, 5, 2, 7, 3]
    t_a, v_a = theta.copy(), v.copy()
    rec_a = oracle.merge_fragment(t_a, v_a, learners, tokens, mask, 2, 0.7, 0.9, steps=steps)
    perm = [4, 0, 5, 2, 1, 3]                      # new position j holds old learner perm[j]
    mask_p = sum(((mask >> perm[j]) & 1) << j for j in range(M))
    t_b, v_b = theta.copy(), v.copy()
    rec_b = oracle.merge_fragment(t_b, v_b, [learners[p] for p in perm],
                                  [tokens[p] for p in perm], mask_p, 2, 0.7, 0.9,
                                  steps=[steps[p] for p in perm])
    assert sorted(perm[j] for j in rec_b.idx) == rec_a.idx
    np.testing.assert_allclose(t_b, t_a, rtol=1e-6, atol=1e-10)
    np.testing.assert_allclose(v_b, v_a, rtol=1e-6, atol=1e-10)
    wa = dict(zip(rec_a.idx, rec_a.w_hat))
    for j, w in zip(rec_b.idx, rec_b.w_hat):
        assert math.isclose(w, wa[perm[j]], rel_tol=1e-14)


# ---- algebra of the outer step ----------------------------------------------------

@pytest.mark.parametrize("nesterov", [True, False])
def test_zero_outer_gradient(nesterov):
    n = 1000
    rng = np.random.default_rng(4)
    theta = rng.normal(0, 0.02, n).astype(np.float32)
    v = rng.normal(0, 1e-3, n).astype(np.float32)
    learners = [theta.copy(), theta.copy(), theta.copy()]
    eta, mu = np.float32(0.7), np.float32(0.9)
    t0, v0 = theta.astype(np.float64), v.astype(np.float64)
    rec = oracle.merge_fragment(theta, v, learners, [3, 4, 5], 0b111, 3, eta, mu,
                                nesterov=nesterov)
    mu_d, eta_d = float(mu), float(eta)
    np.testing.assert_allclose(v, mu_d * v0, rtol=1e-7)
    step = eta_d * mu_d * mu_d * v0 if nesterov else eta_d * mu_d * v0
    np.testing.assert_allclose(theta, t0 - step, rtol=1e-7, atol=1e-12)
    assert rec.delta_sq == 0.0 and all(x == 0.0 for x in rec.delta_m_sq)


def test_single_participant_copies_learner_when_lr1():
    theta, v, learners = _frag(M=3, seed=9)
    rec = oracle.merge_fragment(theta, v, learners, [9, 9, 9], 0b010, 1, 1.0, 0.0)
    assert rec.idx == [1] and rec.w_hat == [1.0]
    np.testing.assert_array_equal(theta, learners[1])


def test_token_scaling():
    theta, v, learners = _frag(M=4, dtype="bf16", seed=12)
    tokens = [1234, 999, 31337, 4242]
    t_a, v_a = theta.copy(), v.copy()
    rec_a = oracle.merge_fragment(t_a, v_a, learners, tokens, 0b1111, 1, 0.7, 0.9)
    t_b, v_b = theta.copy(), v.copy()
    rec_b = oracle.merge_fragment(t_b, v_b, learners, [t * 1024 for t in tokens], 0b1111, 1,
                                  0.7, 0.9)
    assert rec_a.w_hat == rec_b.w_hat                 # powers of two: bit-identical
    np.testing.assert_array_equal(t_a, t_b)
    np.testing.assert_array_equal(v_a, v_b)
    t_c, v_c = theta.copy(), v.copy()
    rec_c = oracle.merge_fragment(t_c, v_c, learners, [t * 3 for t in tokens], 0b1111, 1, 0.7, 0.9)
    np.testing.assert_allclose(rec_c.w_hat, rec_a.w_hat, rtol=1e-15)
    np.testing.assert_allclose(t_c, t_a, rtol=1e-6)


def test_weight_is_tokens_squared_over_steps():
    tokens = [4000, 9000, 100, 2500]
    steps = [4, 3, 1, 5]
    st, w_hat, W = oracle.weights(tokens, steps, [0, 1, 3])
    raw = [tokens[m] * (tokens[m] / steps[m]) for m in (0, 1, 3)]
    assert st == 0 and math.isclose(W, sum(raw), rel_tol=1e-15)
    np.testing.assert_allclose(w_hat, np.array(raw) / sum(raw), rtol=1e-15)
    assert math.isclose(sum(w_hat), 1.0, rel_tol=1e-15)
    # fewer steps for the same tokens -> larger weight ("quality")
    _, w2, _ = oracle.weights([1000, 1000], [10, 5], [0, 1])
    assert math.isclose(w2[1] / w2[0], 2.0, rel_tol=1e-15)
    with pytest.raises(ValueError):
        oracle.weights([10, 10], [1, 0], [0, 1])


def test_constant_tokens_per_step_equals_token_weights():
    theta, v, learners = _frag(M=4, seed=13)
    steps = [3, 7, 1, 12]
    tokens = [4096 * s for s in steps]              # same batch size everywhere
    t_a, v_a = theta.copy(), v.copy()
    rec_a = oracle.merge_fragment(t_a, v_a, learners, tokens, 0b1111, 1, 0.7, 0.9)
    t_b, v_b = theta.copy(), v.copy()
    rec_b = oracle.merge_fragment(t_b, v_b, learners, tokens, 0b1111, 1, 0.7, 0.9, steps=steps)
    np.testing.assert_allclose(rec_b.w_hat, rec_a.w_hat, rtol=1e-15)
    np.testing.assert_allclose(t_b, t_a, rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(v_b, v_a, rtol=1e-6, atol=1e-12)


@pytest.mark.parametrize("nesterov", [True, False])
def test_two_merge_momentum_recurrence(nesterov):
    # The same outer gradient D twice from v0 = 0:
    #   Nesterov:   v1 = D, T1 = T0 - eta (1+mu) D ; v2 = (1+mu) D,
    #               T2 = T0 - eta D [(1+mu) + (1+mu+mu^2)]
    #   heavy ball: T1 = T0 - eta D ; T2 = T0 - eta D (2+mu)
    n = 512
    rng = np.random.default_rng(21)
    theta = rng.normal(0, 0.02, n).astype(np.float32)
    D = rng.normal(0, 1e-3, n).astype(np.float32).astype(np.float64)
    v = np.zeros(n, dtype=np.float32)
    eta, mu = 0.5, 0.75                                # exact in binary
    T0 = theta.astype(np.float64)
    for k in (1, 2):
        learners = [(theta.astype(np.float64) - D).astype(np.float32)] * 2
        d_actual = np.mean([theta.astype(np.float64) - a.astype(np.float64) for a in learners],
                           axis=0)
        np.testing.assert_allclose(d_actual, D, rtol=1e-4, atol=1e-9)
        oracle.merge_fragment(theta, v, learners, [1, 1], 0b11, 2, eta, mu, nesterov=nesterov)
        if k == 1:
            c_v, c_t = 1.0, ((1 + mu) if nesterov else 1.0)
        else:
            c_v = 1 + mu
            c_t = ((1 + mu) + (1 + mu + mu * mu)) if nesterov else (2 + mu)
        np.testing.assert_allclose(v, c_v * D, rtol=2e-4, atol=1e-9)
        np.testing.assert_allclose(theta, T0 - eta * c_t * D, rtol=1e-6, atol=2e-7)


def test_outer_step_matches_torch_sgd():
    # Independent third implementation: torch.optim.SGD fed grad = Delta.
    theta, v, learners = _frag(n=2048, M=4, dtype="bf16", seed=17)
    tokens = [1000, 3000, 2000, 500]
    w = torch.tensor(tokens, dtype=torch.float64) / sum(tokens)
    for nesterov in (True, False):
        p = torch.nn.Parameter(torch.from_numpy(theta.copy()).double())
        opt = torch.optim.SGD([p], lr=0.7, momentum=0.9, nesterov=nesterov, dampening=0.0)
        t_o, v_o = theta.copy(), v.copy()
        for _ in range(3):                            # momentum buffer carried across merges
            L = torch.stack([torch.from_numpy(_as_f64(a)) for a in learners])
            p.grad = (w[:, None] * (p.detach()[None, :] - L)).sum(0)
            opt.step()
            oracle.merge_fragment(t_o, v_o, learners, tokens, 0b1111, 4, 0.7, 0.9,
                                  nesterov=nesterov)
            # eta, mu are widened from float32 in the oracle: 0.7f != 0.7
            np.testing.assert_allclose(t_o, p.detach().numpy(), rtol=3e-6, atol=3e-8)
        buf = opt.state[p]["momentum_buffer"].numpy()
        np.testing.assert_allclose(v_o, buf, rtol=1e-5, atol=1e-8)


# ---- norm diagnostics ("near-orthogonal outer gradients of norm R average to R/sqrt(M)")

def test_norm_statistics_of_iid_outer_gradients():
    n, M = 1 << 18, 8
    theta, v, learners = synth.fragment_cpu(n, M, "f32", seed=31)
    tokens = [100, 200, 300, 400, 500, 600, 700, 800]
    rec = oracle.merge_fragment(theta, v, learners, tokens, _full_mask(M), M, 0.7, 0.9)
    sigma2 = synth.LEARNER_NOISE_STD ** 2
    tol = 6.0 * math.sqrt(2.0 / n)                    # chi-square relative spread, 6 sigma
    for x in rec.delta_m_sq:
        assert abs(x / (n * sigma2) - 1.0) < tol
    sum_w2 = sum(w * w for w in rec.w_hat)
    assert abs(rec.delta_sq / (n * sigma2 * sum_w2) - 1.0) < tol
    # equal weights: ||Delta|| ~ R / sqrt(M)
    theta, v, learners = synth.fragment_cpu(n, M, "f32", seed=32)
    rec = oracle.merge_fragment(theta, v, learners, [5] * M, _full_mask(M), M, 0.7, 0.9)
    R = math.sqrt(np.mean(rec.delta_m_sq))
    assert abs(math.sqrt(rec.delta_sq) / (R / math.sqrt(M)) - 1.0) < tol
    np.testing.assert_allclose(rec.theta_sq, float(np.sum(theta.astype(np.float64) ** 2)),
                               rtol=1e-12)
    np.testing.assert_allclose(rec.mom_sq, float(np.sum(v.astype(np.float64) ** 2)), rtol=1e-12)


# ---- participation: brute force -----------------------------------------------------

def test_participants_brute_force():
    for M in (1, 2, 3, 4):
        for tokens in itertools.product((0, 1, 5), repeat=M):
            for mask in range(1 << M):
                expect = [m for m in range(M) if (mask >> m) & 1 and tokens[m] > 0]
                for K in range(M + 1):
                    st, idx = oracle.participants(mask, list(tokens), K)
                    assert idx == expect
                    assert st == (0 if len(expect) >= max(K, 1) else 1)


def test_participants_wide_and_high_bits():
    M = 64
    tokens = [1] * M
    st, idx = oracle.participants(1 << 63, tokens, 1)
    assert st == 0 and idx == [63]
    st, idx = oracle.participants((1 << 64) - 1, tokens, 64)
    assert st == 0 and idx == list(range(64))
    # bits at positions >= M are ignored
    st, idx = oracle.participants(0b11111000, [3, 3, 3], 1)
    assert st == 1 and idx == []
    with pytest.raises(ValueError):
        oracle.participants(1, [1] * 65, 1)
    with pytest.raises(ValueError):
        oracle.participants(1, [1, 1], 3)


# ---- grace window -----------------------------------------------------------------

def test_grace_window_closed_form():
    # slack = tau * step - (quorum + sync); grace = gamma * slack, never negative
    assert oracle.grace_window(2.0, 1.0, 0.25, 0.5, 0.5) == 0.5 * (2.0 - 0.75)
    assert oracle.grace_window(2.0, 3.0, 1.0, 1.0, 0.25) == 1.0
    assert oracle.grace_window(2.0, 1.0, 1.5, 1.0, 0.9) == 0.0
    assert oracle.grace_window(1.0, 1.0, 0.5, 0.5, 0.9) == 0.0


def _select_restatement(arrival, K, grace):
    fin = sorted(a for a in arrival if math.isfinite(a))
    K = max(K, 1)
    if len(fin) < K:
        return 1, 0, 0
    deadline = fin[K - 1] + grace
    members = [m for m, a in enumerate(arrival) if a <= deadline]
    return 0, sum(1 << m for m in members), len(members)


def test_select_quorum_against_sort_restatement():
    rng = np.random.default_rng(8)
    for trial in range(400):
        M = int(rng.integers(1, 13))
        arrival = rng.integers(0, 6, size=M).astype(float) * 0.25      # many ties
        arrival[rng.random(M) < 0.2] = math.inf
        K = int(rng.integers(0, M + 1))
        grace = float(rng.choice([0.0, 0.25, 0.3, 1.0]))
        assert oracle.select_quorum(arrival.tolist(), K, grace) == \
            _select_restatement(arrival.tolist(), K, grace)


def test_select_quorum_examples():
    # K = 2 of 4; the third report lands inside the grace window, the fourth never comes
    assert oracle.select_quorum([0.1, 0.5, math.inf, 0.2], 2, 0.0) == (0, 0b1001, 2)
    assert oracle.select_quorum([0.1, 0.5, math.inf, 0.2], 2, 0.3) == (0, 0b1011, 3)
    assert oracle.select_quorum([0.1, math.inf, math.inf, math.inf], 2, 10.0) == (1, 0, 0)


def test_grace_recipe_admits_13_of_16():
    w = synth.workload("dense1b3")
    st, mask, n_adm = oracle.select_quorum(w.arrival_s.tolist(), w.K, w.grace_s)
    assert st == 0 and n_adm == 13 and mask == w.masks[0]
    st, _, n0 = oracle.select_quorum(w.arrival_s.tolist(), w.K, 0.0)
    assert n0 == w.K


# ---- bf16 rounding ----------------------------------------------------------------

def test_bf16_rne_matches_torch_cast():
    upper = np.arange(1 << 16, dtype=np.uint32) << 16
    for lower in (0x0000, 0x0001, 0x7fff, 0x8000, 0x8001, 0xffff, 0x4000, 0xc000):
        bits = (upper | np.uint32(lower)).astype(np.uint32)
        x = bits.view(np.float32)
        got = oracle.bf16_rne(x)
        ref = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        nan = np.isnan(x)
        np.testing.assert_array_equal(got[~nan], ref[~nan])
        assert np.all(np.isnan(oracle.bf16_to_f32(got[nan])))


def test_bf16_output_is_rounded_state():
    theta, v, learners = _frag(M=3, dtype="bf16", seed=23)
    out = np.zeros(theta.size, dtype=np.uint16)
    oracle.merge_fragment(theta, v, learners, [3, 4, 5], 0b111, 3, 0.7, 0.9, out_bf16=out)
    ref = torch.from_numpy(theta).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(out, ref)


# ---- radial-directional averaging ---------------------------------------------------

def _rda_inputs(vs, theta):
    return [(theta.astype(np.float64) - d).astype(np.float32) for d in vs]


def test_rda_equal_norms_keep_norm():
    # ||v_i|| = R for all i  =>  ||RDA|| = R
    n, M, R = 4096, 5, 0.37
    rng = np.random.default_rng(41)
    theta = np.zeros(n, dtype=np.float32)
    vs = []
    for _ in range(M):
        d = rng.normal(size=n)
        vs.append(R * d / np.linalg.norm(d))
    v = np.zeros(n, dtype=np.float32)
    rec = oracle.merge_fragment(theta, v, _rda_inputs(vs, theta), [10, 20, 30, 40, 50],
                                _full_mask(M), M, 1.0, 0.0, merge=oracle.MERGE_RDA)
    assert abs(math.sqrt(rec.delta_sq) / R - 1.0) < 1e-6
    # while the plain average shrinks towards R / sqrt(M)
    theta2, v2 = np.zeros(n, dtype=np.float32), np.zeros(n, dtype=np.float32)
    rec2 = oracle.merge_fragment(theta2, v2, _rda_inputs(vs, theta2), [10] * M, _full_mask(M), M,
                                 1.0, 0.0)
    assert abs(math.sqrt(rec2.delta_sq) / (R / math.sqrt(M)) - 1.0) < 0.1


def test_rda_single_and_collinear():
    n = 1024
    rng = np.random.default_rng(42)
    theta = np.zeros(n, dtype=np.float32)
    d = rng.normal(0, 1e-2, n)
    # s = 1: RDA(v1) = v1
    v = np.zeros(n, dtype=np.float32)
    oracle.merge_fragment(theta, v, _rda_inputs([d], theta), [7], 1, 1, 1.0, 0.0,
                          merge=oracle.MERGE_RDA)
    np.testing.assert_allclose(v, d.astype(np.float32), rtol=1e-6, atol=1e-12)
    # collinear (positive multiples): RDA = weighted mean of the vectors
    theta = np.zeros(n, dtype=np.float32)
    v = np.zeros(n, dtype=np.float32)
    scales, tokens = [1.0, 2.0, 4.0], [100, 300, 600]
    oracle.merge_fragment(theta, v, _rda_inputs([c * d for c in scales], theta), tokens, 0b111, 3,
                          1.0, 0.0, merge=oracle.MERGE_RDA)
    wm = sum(t * c for t, c in zip(tokens, scales)) / sum(tokens)
    np.testing.assert_allclose(v, (wm * d).astype(np.float32), rtol=2e-6, atol=1e-12)


def test_rda_matches_definition():
    n, M = 2048, 4
    theta, v, learners = _frag(n=n, M=M, seed=43)
    tokens = [5, 1, 3, 2]
    w = np.array(tokens, dtype=np.float64) / sum(tokens)
    T = theta.astype(np.float64)
    ds = [T - _as_f64(a) for a in learners]
    norms = [np.linalg.norm(x) for x in ds]
    u = sum(w[m] * ds[m] / norms[m] for m in range(M))
    expect = sum(w[m] * norms[m] for m in range(M)) * u / np.linalg.norm(u)
    oracle.merge_fragment(theta, v, learners, tokens, _full_mask(M), M, 1.0, 0.0,
                          merge=oracle.MERGE_RDA)
    np.testing.assert_allclose(v, expect.astype(np.float32), rtol=1e-5, atol=1e-10)


# ---- learner side: theta <- alpha theta + (1 - alpha) Theta ---------------------------

def test_apply_to_learner_special_cases():
    theta, _, learners = _frag(n=3000, M=2, dtype="bf16", seed=51)
    before = learners[0].copy()
    # alpha = 0 (the paper's choice): a plain overwrite with the rounded global fragment
    oracle.apply_to_learner(learners[0], theta, 0.0)
    ref = torch.from_numpy(theta).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(learners[0], ref)
    # alpha = 1: the learner keeps its copy
    oracle.apply_to_learner(learners[1], theta, 1.0)
    _, _, again = _frag(n=3000, M=2, dtype="bf16", seed=51)
    np.testing.assert_array_equal(learners[1], again[1])
    # alpha = 1/2 in float32: the midpoint
    t32, _, l32 = _frag(n=3000, M=1, dtype="f32", seed=52)
    mid = (0.5 * l32[0].astype(np.float64) + 0.5 * t32.astype(np.float64)).astype(np.float32)
    oracle.apply_to_learner(l32[0], t32, 0.5)
    np.testing.assert_array_equal(l32[0], mid)
    assert not np.array_equal(before, learners[0])


def test_grace_controller_moving_average_closed_form():
    # constant observations: averages stay put; a step change decays geometrically
    w = oracle.grace_controller_window(2.0, 0.5, 0.9, [(1.0, 0.2, 0.3)] * 7)
    assert math.isclose(w, 0.5 * (2.0 * 1.0 - 0.5), rel_tol=1e-12)
    obs = [(1.0, 0.0, 0.0)] + [(2.0, 0.0, 0.0)] * 5
    xi = 2.0 - 0.9 ** 5                         # 1 -> 2 with beta = 0.9 after 5 updates
    assert math.isclose(oracle.grace_controller_window(1.0, 0.5, 0.9, obs), 0.5 * xi, rel_tol=1e-12)
    assert oracle.grace_controller_window(2.0, 0.5, 0.9, []) == 0.0


# ---- a merge worked by hand (tests/golden/merge_hand_worked.txt) -------------------------

def _hand_worked():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "merge_hand_worked.txt")
    out = {}
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            key, *vals = line.split()
            out[key] = [float(x) for x in vals]
    return out


def test_hand_worked_merge():
    g = _hand_worked()
    tokens = [int(t) for t in g["tokens"]]
    for nesterov, key in ((True, "theta_nesterov"), (False, "theta_heavy")):
        theta = np.array(g["theta"], dtype=np.float32)
        v = np.array(g["momentum"], dtype=np.float32)
        learners = [np.array(g["learner0"], dtype=np.float32), np.array(g["learner1"], dtype=np.float32)]
        rec = oracle.merge_fragment(theta, v, learners, tokens, 0b11, 2, g["eta"][0], g["mu"][0],
                                    nesterov=nesterov)
        assert rec.w_hat == g["w_hat"]
        np.testing.assert_array_equal(v, np.array(g["momentum_new"], dtype=np.float32))
        np.testing.assert_array_equal(theta, np.array(g[key], dtype=np.float32))
        assert rec.delta_sq == g["delta_sq"][0] and rec.delta_m_sq == g["delta_m_sq"]
    # radial-directional merge of the same inputs, from the closed form in the fixture's header
    theta = np.array(g["theta"], dtype=np.float32)
    v = np.zeros(2, dtype=np.float32)
    learners = [np.array(g["learner0"], dtype=np.float32), np.array(g["learner1"], dtype=np.float32)]
    oracle.merge_fragment(theta, v, learners, tokens, 0b11, 2, 1.0, 0.0, merge=oracle.MERGE_RDA)
    s5 = math.sqrt(5.0)
    d = np.array([0.25 * 1 + 0.75 * (-1) / s5, 0.75 * 2 / s5])
    expect = (0.25 + 0.75 * s5) * d / np.linalg.norm(d)
    np.testing.assert_allclose(v, expect.astype(np.float32), rtol=1e-6)


def test_huge_token_counts():
    # counts far beyond 2^53: the integer sum stays exact, the weights stay normalised
    big = [2**62, 2**61, 2**61 + 12345]
    st, w_hat, W = oracle.weights(big, None, [0, 1, 2])
    assert st == 0 and W == float(sum(big))
    np.testing.assert_allclose(w_hat, [b / sum(big) for b in big], rtol=1e-15)
    with pytest.raises(ValueError):
        oracle.weights([2**63, 2**63], None, [0, 1])        # the exact sum would wrap


def test_rda_stages_equal_the_whole_merge_and_add_up_over_ranges():
    # one range: the three stages ARE the merge, bit for bit; three ranges with the stage outputs
    # summed in between: the same merge up to the order of the sums
    n, M = 3001, 4
    theta, v, learners = _frag(n=n, M=M, dtype="bf16", seed=55)
    v[:] = np.random.default_rng(3).normal(0, 1e-3, n).astype(np.float32)
    tokens, mask, K = [5, 0, 2, 9], 0b1101, 2
    t_ref, v_ref = theta.copy(), v.copy()
    ref = oracle.merge_fragment(t_ref, v_ref, learners, tokens, mask, K, 0.7, 0.9, merge=oracle.MERGE_RDA)
    t1, v1 = theta.copy(), v.copy()
    r0, _ = oracle.merge_fragment_rda_stage(0, t1, v1, learners, tokens, mask, K, 0.7, 0.9)
    _, d = oracle.merge_fragment_rda_stage(1, t1, v1, learners, tokens, mask, K, 0.7, 0.9, norms_sq=r0.delta_m_sq)
    r2, _ = oracle.merge_fragment_rda_stage(2, t1, v1, learners, tokens, mask, K, 0.7, 0.9,
                                            norms_sq=r0.delta_m_sq, dir_sq=d)
    np.testing.assert_array_equal(t1, t_ref)
    np.testing.assert_array_equal(v1, v_ref)
    assert (r2.delta_sq, r2.theta_sq, r2.mom_sq, r0.delta_m_sq) == (ref.delta_sq, ref.theta_sq, ref.mom_sq, ref.delta_m_sq)
    cuts = [(0, 1000), (1000, 1008), (1008, n)]
    shard = [(theta[a:b].copy(), v[a:b].copy(), [x[a:b].copy() for x in learners]) for a, b in cuts]
    norms = np.sum([oracle.merge_fragment_rda_stage(0, t, m, l, tokens, mask, K, 0.7, 0.9)[0].delta_m_sq
                    for t, m, l in shard], axis=0)
    dsq = sum(oracle.merge_fragment_rda_stage(1, t, m, l, tokens, mask, K, 0.7, 0.9, norms_sq=norms)[1]
              for t, m, l in shard)
    recs = [oracle.merge_fragment_rda_stage(2, t, m, l, tokens, mask, K, 0.7, 0.9, norms_sq=norms, dir_sq=dsq)[0]
            for t, m, l in shard]
    np.testing.assert_allclose(np.concatenate([t for t, _, _ in shard]), t_ref, rtol=0, atol=2e-9)
    np.testing.assert_allclose(np.concatenate([m for _, m, _ in shard]), v_ref, rtol=0, atol=1e-9)
    assert abs(sum(r.delta_sq for r in recs) - ref.delta_sq) <= 1e-12 * ref.delta_sq
    # the stage interface refuses a later stage without the summed output of the earlier one
    with pytest.raises(ValueError):
        oracle.merge_fragment_rda_stage(1, t1, v1, learners, tokens, mask, K, 0.7, 0.9)


# ---- int4 compression of outer gradients (reading of this build; the paper gives no quantiser) ----

def test_int4_quantiser_properties():
    n = 1000                                           # 7 full blocks of 128 and a ragged one
    theta, _, learners = _frag(n=n, M=2, dtype="bf16", seed=71)
    codes, scales = oracle.quantize_int4(theta, learners[0])
    d = theta - oracle.bf16_to_f32(learners[0])        # float32 differences
    nib = np.concatenate([codes & 15, codes >> 4]).reshape(2, -1).T.reshape(-1)[:n]
    assert nib.min() >= 1 and nib.max() <= 15          # codes -7..7 stored as code + 8
    dq = oracle.dequantize_int4(codes, scales, n)
    for b in range(len(scales)):
        blk = slice(128 * b, min(n, 128 * (b + 1)))
        amax = np.max(np.abs(d[blk]))
        assert scales[b] == np.float32(amax) / np.float32(7.0)
        # nearest-code rounding: error at most half a step; the largest element is hit exactly
        assert np.max(np.abs(dq[blk] - d[blk])) <= 0.5 * scales[b] * (1 + 1e-6)
        k = np.argmax(np.abs(d[blk]))
        assert abs(int(nib[blk][k]) - 8) == 7
    # quantising an already quantised gradient changes nothing
    learner2 = (theta.astype(np.float64) - dq.astype(np.float64)).astype(np.float32)
    d2 = theta - learner2
    if np.array_equal(d2, dq):                         # only when Theta - (Theta - dq) is exact
        codes2, scales2 = oracle.quantize_int4(theta, learner2)
        np.testing.assert_array_equal(codes2, codes)
    # an all-zero block has scale 0 and code 0 everywhere
    codes0, scales0 = oracle.quantize_int4(theta, theta.copy())
    assert np.all(scales0 == 0) and np.all((codes0 & 15) == 8) and np.all((codes0[: n // 2] >> 4) == 8)
    # ties round to even: d / scale = 2.5 -> 2, 3.5 -> 4
    t = np.zeros(128, dtype=np.float32)
    l = np.zeros(128, dtype=np.float32)
    l[0], l[1], l[2] = -7.0, -2.5, -3.5                # d = 7 (scale 1), 2.5, 3.5
    c, s_ = oracle.quantize_int4(t, l)
    assert s_[0] == 1.0 and (c[0] & 15) == 15 and (c[0] >> 4) == 10 and (c[1] & 15) == 12


def test_int4_quantiser_non_finite_differences_poison_their_block():
    # three blocks: a NaN, an infinity, and an ordinary one that must be untouched by its neighbours
    t = np.zeros(384, dtype=np.float32)
    l = np.full(384, -1.0, dtype=np.float32)
    l[3] = np.nan
    l[128 + 7] = -np.inf                                # d = +inf
    l[128 + 8] = np.inf                                 # d = -inf
    c, s_ = oracle.quantize_int4(t, l)
    assert np.isnan(s_[0]) and np.isposinf(s_[1]) and s_[2] == np.float32(1.0) / np.float32(7.0)
    nib = np.stack([c & 15, c >> 4], axis=1).reshape(-1)
    assert np.all(nib[:128] == 8)                       # NaN scale: every code 0
    assert nib[128 + 7] == 1 and nib[128 + 8] == 1      # inf / inf is NaN, coded -7
    assert np.all(np.delete(nib[128:256], [7, 8]) == 8) # finite / inf = 0
    assert np.all(nib[256:] == 15)                      # the ordinary block: d = 1 = 7 * scale
    dq = oracle.dequantize_int4(c, s_, 384)
    assert not np.isfinite(dq[:256]).any() and np.all(dq[256:] == np.float32(7.0) * s_[2])


def test_int4_merge_equals_plain_merge_of_dequantised_gradients():
    n, M = 3000, 4
    theta, v, learners = _frag(n=n, M=M, dtype="bf16", seed=72)
    v[:] = np.random.default_rng(1).normal(0, 1e-3, n).astype(np.float32)
    tokens, mask = [10, 0, 30, 40], 0b1101
    q = [oracle.quantize_int4(theta, a) for a in learners]
    # a learner whose copy IS Theta - D^ reproduces the compressed gradient (up to one float32 rounding)
    recon = [(theta.astype(np.float64) - oracle.dequantize_int4(c, s_, n)).astype(np.float32) for c, s_ in q]
    t_a, v_a = theta.copy(), v.copy()
    ra = oracle.merge_fragment_int4(t_a, v_a, [c for c, _ in q], [s_ for _, s_ in q], tokens, mask, 2,
                                    0.7, 0.9)
    t_b, v_b = theta.copy(), v.copy()
    rb = oracle.merge_fragment(t_b, v_b, recon, tokens, mask, 2, 0.7, 0.9)
    assert ra.idx == rb.idx == [0, 2, 3] and ra.w_hat == rb.w_hat
    np.testing.assert_allclose(v_a, v_b, rtol=0, atol=2e-9)
    np.testing.assert_allclose(t_a, t_b, rtol=0, atol=1.5e-8)          # an ulp of Theta at 0.1
    # and it stays within half a quantisation step of the uncompressed merge
    t_c, v_c = theta.copy(), v.copy()
    oracle.merge_fragment(t_c, v_c, learners, tokens, mask, 2, 0.7, 0.9)
    step = max(float(np.max(s_)) for _, s_ in q)
    assert np.max(np.abs(v_a - v_c)) <= 0.5 * step * 1.001


def test_all_cores_baseline_agrees_with_the_oracle():
    # the OpenMP loop is only a timing baseline, but it must compute the same merge
    theta, v, learners = _frag(n=50_001, M=5, dtype="bf16", seed=81)
    tokens, mask = [10, 20, 0, 40, 50], 0b11101
    t_a, v_a = theta.copy(), v.copy()
    ref = oracle.merge_fragment(t_a, v_a, learners, tokens, mask, 2, 0.7, 0.9)
    t_b, v_b = theta.copy(), v.copy()
    dsq = oracle.merge_fragment_all_cores(t_b, v_b, learners, tokens, mask, 2, 0.7, 0.9)
    np.testing.assert_array_equal(t_a, t_b)
    np.testing.assert_array_equal(v_a, v_b)
    assert abs(dsq - ref.delta_sq) <= 1e-12 * ref.delta_sq
    assert oracle.merge_fragment_all_cores(t_b, v_b, learners, tokens, mask, 5, 0.7, 0.9) is None
