"""Oracle for the fragmentation strategies (TEST INFRASTRUCTURE ONLY).

Plain-Python statements of the three strategies of the appendix "Fragmentation
strategies", plus a brute-force optimal partition for tiny inputs.  Shares nothing
with the library's planner.

Pins (tests/test_fragmentation.py): the two worked index examples the paper
prints (tests/golden/fragmentation_examples.txt), the 4/3 bound of greedy number
partitioning against the brute-force optimum, and partition invariants.
"""
from __future__ import annotations

import itertools


def layer_fragments(layer, P):
    """One fragment for all non-transformer tensors (layer < 0); transformer
    layers are dealt out to the other P - 1 fragments by strided selection."""
    buckets = P - 1
    return [0 if l < 0 else 1 + l % buckets for l in layer]


def tensor_fragments(layer, P):
    """As above, but strided over the running index of the transformer tensors."""
    buckets = P - 1
    out, i = [], 0
    for l in layer:
        if l < 0:
            out.append(0)
        else:
            out.append(1 + i % buckets)
            i += 1
    return out


def balanced_fragments(size_bits, P):
    """Greedy number partitioning: tensors in descending size, each into the
    currently smallest fragment."""
    totals = [0] * P
    out = [None] * len(size_bits)
    for q in sorted(range(len(size_bits)), key=lambda q: (-size_bits[q], q)):
        p = min(range(P), key=lambda p: (totals[p], p))
        out[q] = p
        totals[p] += size_bits[q]
    return out


def optimal_peak(size_bits, P):
    """Smallest possible largest-fragment size, by exhaustive search (tiny Q only)."""
    best = None
    for assign in itertools.product(range(P), repeat=len(size_bits)):
        totals = [0] * P
        for q, p in enumerate(assign):
            totals[p] += size_bits[q]
        peak = max(totals)
        if best is None or peak < best:
            best = peak
    return best
