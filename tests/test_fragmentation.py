"""Fragmentation planner: oracle against the paper's worked examples and the
mathematics, and the library's planner against the oracle."""
import os

import numpy as np
import pytest

from oracle import fragmentation as ofrag

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fragmentation_examples.txt")


@pytest.fixture(scope="module")
def dd():
    from paper_2604_21428_b200 import build
    build.build()
    from paper_2604_21428_b200 import ddmerge
    return ddmerge


def _golden():
    cases = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        kind, items, buckets, frags = [x.strip() for x in line.split("|")]
        groups = [[int(i) for i in g.split(",")] for g in frags.split(";")]
        cases.append((kind, int(items), int(buckets), groups))
    return cases


def _groups(assignment, first_fragment=1):
    out = {}
    for i, p in enumerate(assignment):
        if p >= first_fragment:
            out.setdefault(p, []).append(i + 1)          # 1-based as printed
    return [out[p] for p in sorted(out)]


def test_oracle_reproduces_the_printed_examples():
    cases = _golden()
    assert len(cases) == 2
    for kind, items, buckets, groups in cases:
        if kind == "layer":
            # one tensor per layer plus an embedding that must land in fragment 0
            layer = [-1] + list(range(items))
            got = ofrag.layer_fragments(layer, buckets + 1)
            assert got[0] == 0
            assert _groups(got[1:]) == groups
        else:
            layer = [-1] + [i // 3 for i in range(items)]          # any layer ids: order rules
            got = ofrag.tensor_fragments(layer, buckets + 1)
            assert got[0] == 0
            assert _groups(got[1:]) == groups


def test_layer_strategy_keeps_a_layer_together():
    layer = [-1, 0, 0, 0, 1, 1, 1, 2, 2, 2, 3, 3, 3, -1]
    got = ofrag.layer_fragments(layer, 3)
    for l in range(4):
        assert len({got[i] for i, x in enumerate(layer) if x == l}) == 1
    assert got[0] == got[-1] == 0


def test_greedy_is_within_four_thirds_of_optimal():
    rng = np.random.default_rng(3)
    worst = 0.0
    for trial in range(120):
        Q = int(rng.integers(1, 9))
        P = int(rng.integers(1, 5))
        sizes = [int(x) for x in rng.integers(1, 100, size=Q)]
        assign = ofrag.balanced_fragments(sizes, P)
        totals = [sum(s for s, p in zip(sizes, assign) if p == f) for f in range(P)]
        opt = ofrag.optimal_peak(sizes, P)
        assert sum(totals) == sum(sizes)
        assert max(totals) * 3 <= opt * 4            # Graham's bound for largest-first greedy
        worst = max(worst, max(totals) / opt)
    assert worst >= 1.0
    # the classic tight-ish instance: {3,3,2,2,2} on 2 machines -> greedy 7, optimal 6
    assert ofrag.balanced_fragments([3, 3, 2, 2, 2], 2) == [0, 1, 0, 1, 0]
    assert ofrag.optimal_peak([3, 3, 2, 2, 2], 2) == 6


def test_library_planner_matches_oracle(dd):
    rng = np.random.default_rng(4)
    for trial in range(200):
        L = int(rng.integers(1, 9))
        per_layer = int(rng.integers(1, 7))
        layer = [-1] + [l for l in range(L) for _ in range(per_layer)] + [-1, -1]
        sizes = [int(x) for x in rng.integers(1, 1 << 40, size=len(layer))]
        if trial % 3 == 0:
            sizes = [int(x) for x in rng.integers(1, 4, size=len(layer))]      # many ties
        P_bal = int(rng.integers(1, 26))
        got, totals = dd.plan_fragments(sizes, None, P_bal, dd.FRAG_BALANCED)
        assert got == ofrag.balanced_fragments(sizes, P_bal)
        assert totals == [sum(s for s, p in zip(sizes, got) if p == f) for f in range(P_bal)]
        P = int(rng.integers(2, L + 2))
        got, totals = dd.plan_fragments(sizes, layer, P, dd.FRAG_LAYER)
        assert got == ofrag.layer_fragments(layer, P)
        got, _ = dd.plan_fragments(sizes, layer, P, dd.FRAG_TENSOR)
        assert got == ofrag.tensor_fragments(layer, P)


def test_library_planner_on_the_printed_examples(dd):
    for kind, items, buckets, groups in _golden():
        layer = [-1] + (list(range(items)) if kind == "layer" else [0] * items)
        strategy = dd.FRAG_LAYER if kind == "layer" else dd.FRAG_TENSOR
        got, _ = dd.plan_fragments([8] * len(layer), layer, buckets + 1, strategy)
        assert got[0] == 0 and _groups(got[1:]) == groups


def test_library_planner_rejects_bad_requests(dd):
    with pytest.raises(dd.DDMergeError):
        dd.plan_fragments([1, 2], [0, 1], 4, dd.FRAG_LAYER)       # P - 1 = 3 > 2 layers
    with pytest.raises(dd.DDMergeError):
        dd.plan_fragments([1, 2], [0, 1], 1, dd.FRAG_TENSOR)      # no bucket for transformer tensors
    with pytest.raises(dd.DDMergeError):
        dd.plan_fragments([1, 2], None, 0, dd.FRAG_BALANCED)
    with pytest.raises(dd.DDMergeError):
        dd.plan_fragments([1, 2], [0, 1], 2, 7)
    assert dd.plan_fragments([5, 5], [-1, -1], 1, dd.FRAG_TENSOR)[0] == [0, 0]


def test_balanced_plan_of_a_24_fragment_model(dd):
    # P = H = 24 as in the paper's experiments: a 2B-like dense model's tensor list
    d, ff, V, L = 2048, 8192, 32000, 24
    sizes, layer = [V * d * 16], [-1]
    for l in range(L):
        sizes += [x * 16 for x in (d * d, d * d, d * d, d * d, d * ff, d * ff, d, d)]
        layer += [l] * 8
    sizes += [d * 16, V * d * 16]
    layer += [-1, -1]
    got, totals = dd.plan_fragments(sizes, None, 24, dd.FRAG_BALANCED)
    lower = max(max(sizes), -(-sum(sizes) // 24))       # any packing's peak is at least this
    assert max(totals) * 3 <= lower * 4
    _, t_tensor = dd.plan_fragments(sizes, layer, 24, dd.FRAG_TENSOR)
    assert max(totals) <= max(t_tensor)                 # balancing lowers the peak
