"""The syncer loop replayed from a synthetic event tape: GPU library vs the oracle.

Both sides run Algorithm 2 for the same tape -- quorum with grace window, merge of
the due fragments, broadcast to the learners that are up -- and between syncer
steps every learner copy drifts by the same seeded random walk (a stand-in for
inner optimisation).  State is carried, not resynchronised, so the comparison
allows for the feedback of rounding differences through the outer gradient.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_21428_b200 import synth
from parity_util import floor_rel_err, to_torch_learner

pytestmark = pytest.mark.gpu


def _to_host(t):
    t = t.cpu()
    return t.view(torch.int16).numpy().view(np.uint16).copy() if t.dtype == torch.bfloat16 else t.numpy().copy()


@pytest.mark.parametrize("use_rda,fused", [(False, True), (False, False), (True, True), (True, False)])
def test_replay_matches_oracle(use_rda, fused):
    from paper_2604_21428_b200 import ddmerge as dd
    from paper_2604_21428_b200.replay import Syncer, TapeEntry

    M, P, H, K, T = 5, 4, 4, 2, 14
    sizes = [9_000, 20_011, 4_096, 12_345]
    offsets = [0, 1, 2, 3]
    kinds = [dd.MERGE_AVG] + [dd.MERGE_RDA if use_rda else dd.MERGE_AVG] * (P - 1)
    tape = synth.synthetic_tape(M, P, H, offsets, T, seed=5)
    eta, mu, grace = 0.7, 0.9, 0.25

    h_theta, h_mom, h_learn = [], [], [[None] * P for _ in range(M)]
    for p, n in enumerate(sizes):
        theta, v, learners = synth.fragment_cpu(n, M, "bf16", 800 + p)
        h_theta.append(theta)
        h_mom.append(v)
        for m in range(M):
            h_learn[m][p] = learners[m]
    d_theta = [torch.from_numpy(a.copy()).cuda() for a in h_theta]
    d_mom = [torch.from_numpy(a.copy()).cuda() for a in h_mom]
    d_learn = [[to_torch_learner(h_learn[m][p], "cuda") for p in range(P)] for m in range(M)]

    ctx = dd.Context(0)
    syncer = Syncer(ctx, d_theta, d_mom, H=H, offsets=offsets, K=K, outer_lr=eta, outer_mu=mu,
                    learner_dtype=dd.BF16, merge_kinds=kinds, flags=dd.DIAG_STATE, fused_push=fused)
    drift = np.random.default_rng(17)
    merged = 0
    for t, e in enumerate(tape):
        entry = TapeEntry(arrival_s=e["arrival_s"], tokens=e["tokens"], steps=e["steps"])
        res = syncer.step(t, entry, d_learn, grace_s=grace)
        # ---- the same step with the oracle -------------------------------------------
        st, mask, n_adm = oracle.select_quorum(e["arrival_s"], K, grace)
        assert (res.mask, res.n_admitted) == (mask, n_adm)
        for p, rec in zip(res.due, res.records):
            ref = oracle.merge_fragment(h_theta[p], h_mom[p], [h_learn[m][p] for m in range(M)],
                                        e["tokens"][p], mask, K, eta, mu, steps=e["steps"][p],
                                        merge=oracle.MERGE_RDA if kinds[p] else oracle.MERGE_AVG)
            assert (rec.status, rec.n_part, rec.idx) == (ref.status, ref.n_part, ref.idx), (t, p)
            if ref.status == 0:
                merged += 1
                assert np.allclose(rec.w_hat, ref.w_hat, rtol=1e-6)
                for m in range(M):
                    if math.isfinite(e["arrival_s"][m]):
                        oracle.apply_to_learner(h_learn[m][p], h_theta[p], 0.0)
            # the push reached exactly the learners that are alive (fused into the merge or not)
            for m in range(M):
                same = np.mean(_to_host(d_learn[m][p]) == h_learn[m][p])
                assert same > 0.995, (t, p, m, same)
        # ---- learners move on: identical drift on both sides ---------------------------
        for m in range(M):
            for p, n in enumerate(sizes):
                step = drift.normal(0.0, 3e-4, n).astype(np.float32)
                x = oracle.bf16_to_f32(h_learn[m][p]) + step
                h_learn[m][p] = oracle.bf16_rne(x)
                d_learn[m][p].copy_(to_torch_learner(h_learn[m][p], "cuda"))
    assert merged >= 6
    torch.cuda.synchronize()
    for p in range(P):
        assert floor_rel_err(d_theta[p].cpu().numpy(), h_theta[p]) <= 2e-4, p
        assert float(np.max(np.abs(d_mom[p].cpu().numpy() - h_mom[p]))) <= 2e-7, p
    ctx.close()
