"""Shared helpers for the GPU-vs-oracle parity tests (test code only)."""
from __future__ import annotations

import numpy as np

import oracle

TOL_STATE = 1e-5      # float32 global fragment and momentum
TOL_BF16 = 1e-2       # bf16 broadcast copy
TOL_NORM = 1e-5       # squared-norm diagnostics (relative)


def floor_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |g_i - o_i| / max(|o_i|, rms(o)): relative error with an rms floor.

    A purely element-wise relative error is unbounded at elements that happen to
    be ~0; the floor is the typical magnitude of the array itself.
    """
    got = got.astype(np.float64)
    ref = ref.astype(np.float64)
    if ref.size == 0:
        return 0.0
    nan_g, nan_r = np.isnan(got), np.isnan(ref)
    assert np.array_equal(nan_g, nan_r), "NaN positions differ"
    ok = ~nan_r
    if not ok.any():
        return 0.0
    g, r = got[ok], ref[ok]
    inf = np.isinf(r)
    assert np.array_equal(g[inf], r[inf]), "Inf positions / signs differ"
    g, r = g[~inf], r[~inf]
    if r.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(r * r)))
    denom = np.maximum(np.abs(r), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(g - r) / denom))


def to_torch_learner(a, device):
    import torch
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(a).to(device)


def bf16_bits_to_f32(t) -> np.ndarray:
    """torch bf16 tensor (any device) -> float32 numpy."""
    import torch
    return t.detach().to("cpu").to(torch.float32).numpy()


def assert_record_matches(got, ref, *, diag_state=True, per_learner=True):
    """Integer fields bit-exact; weights bit-exact as float32; norms to TOL_NORM."""
    assert got.status == ref.status, (got.status, ref.status)
    assert got.n_part == ref.n_part
    assert got.idx == ref.idx
    if ref.status != 0:
        assert all(w == 0.0 for w in got.w_hat)
        return
    ref_w = [float(np.float32(w)) for w in ref.w_hat]
    assert got.w_hat == ref_w, (got.w_hat, ref_w)
    assert abs(got.w_total - ref.w_total) <= 1e-12 * abs(ref.w_total)

    def close(a, b):
        return abs(a - b) <= TOL_NORM * abs(b) + 1e-300

    assert close(got.delta_sq, ref.delta_sq), (got.delta_sq, ref.delta_sq)
    if diag_state:
        assert close(got.theta_sq, ref.theta_sq), (got.theta_sq, ref.theta_sq)
        assert close(got.mom_sq, ref.mom_sq), (got.mom_sq, ref.mom_sq)
    else:
        assert got.theta_sq == 0.0 and got.mom_sq == 0.0
    if per_learner:
        for a, b in zip(got.delta_m_sq, ref.delta_m_sq):
            assert close(a, b), (got.delta_m_sq, ref.delta_m_sq)
    else:
        assert all(x == 0.0 for x in got.delta_m_sq)


def oracle_merge(theta, v, learners, tokens, mask, K, eta, mu, **kw):
    return oracle.merge_fragment(theta, v, learners, tokens, mask, K, eta, mu, **kw)
