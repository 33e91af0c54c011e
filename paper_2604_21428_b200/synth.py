"""Seeded synthetic inputs for the per-fragment merge.

This module only draws inputs: fragment shapes, token / step counters, quorum
masks, arrival times and the random parameter values themselves.  It holds none
of the merge's arithmetic and is the one module the tests use on both the CPU
oracle side and the CUDA side.

Recipe (all workloads): the global fragment is N(0, 0.02^2) in fp32; learner m's
copy is global + N(0, (1e-3)^2), formed in fp32 and then rounded to the learner
dtype; the outer momentum starts at zero; counters and masks come from
``numpy.random.default_rng(seed)`` on the host.  Fragments are flat
concatenations of the tensors of a decoder block group: a dense layer is
4 d^2 (q, k, v, o) + 2 d d_ff (up, down) + 2 d (norm gains); the embedding V d
goes into the first fragment, the final norm d and an untied head V d into the
last.  An MoE layer replaces the MLP by E experts of 2 d d_ff plus a d x E router.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

THETA_STD = 0.02
LEARNER_NOISE_STD = 1e-3
OUTER_LR = 0.7
OUTER_MU = 0.9


@dataclass
class Workload:
    name: str
    M: int                       # learners
    K: int                       # minimum quorum
    learner_dtype: str           # "f32" | "bf16"
    fragment_sizes: list         # elements per fragment
    tokens: np.ndarray           # uint64 [P, M]
    masks: list                  # python ints, one per fragment
    seed: int
    repeats: int = 1             # back-to-back merges for steady state
    arrival_s: np.ndarray | None = None
    grace_s: float | None = None
    notes: str = ""
    steps: np.ndarray | None = None

    @property
    def P(self) -> int:
        return len(self.fragment_sizes)

    @property
    def total_params(self) -> int:
        return int(sum(self.fragment_sizes))


def dense_layer_params(d: int, d_ff: int) -> int:
    return 4 * d * d + 2 * d * d_ff + 2 * d


def moe_layer_params(d: int, d_ff: int, experts: int) -> int:
    return 4 * d * d + experts * 2 * d * d_ff + d * experts + 2 * d


def dense_fragments(layers: int, d: int, d_ff: int, vocab: int, P: int) -> list:
    """P contiguous layer groups; embedding in the first, final norm + head in the last."""
    assert layers % P == 0
    per = (layers // P) * dense_layer_params(d, d_ff)
    sizes = [per] * P
    sizes[0] += vocab * d
    sizes[-1] += d + vocab * d
    return sizes


def moe_fragments(layers: int, d: int, d_ff: int, experts: int, vocab: int) -> list:
    """One fragment per layer (ragged: first and last carry embedding / head)."""
    sizes = [moe_layer_params(d, d_ff, experts)] * layers
    sizes[0] += vocab * d
    sizes[-1] += d + vocab * d
    return sizes


def _mask_of(members) -> int:
    mask = 0
    for m in members:
        mask |= 1 << int(m)
    return mask


def workload(name: str) -> Workload:
    """The five named workloads (tiny, dense150m, dense1b3, moe4b, scale500m)."""
    if name == "tiny":
        return Workload(name, M=2, K=2, learner_dtype="f32", fragment_sizes=[1 << 20],
                        tokens=np.array([[1000, 3000]], dtype=np.uint64), masks=[0b11], seed=0)
    if name == "dense150m":
        rng = np.random.default_rng(1)
        sizes = dense_fragments(12, 768, 3072, 32000, 4)
        M = 8
        failed = rng.choice(M, size=2, replace=False)
        mask = _mask_of(m for m in range(M) if m not in set(failed.tolist()))
        tokens = rng.integers(100_000, 300_001, size=(len(sizes), M)).astype(np.uint64)
        return Workload(name, M=M, K=6, learner_dtype="bf16", fragment_sizes=sizes,
                        tokens=tokens, masks=[mask] * len(sizes), seed=1,
                        notes="2 of 8 learners failed")
    if name == "dense1b3":
        rng = np.random.default_rng(2)
        sizes = dense_fragments(24, 2048, 8192, 32000, 8)
        M, K, admit = 16, 8, 13
        arrival = rng.lognormal(mean=0.0, sigma=0.5, size=M)
        order = np.sort(arrival)
        grace = 0.5 * (order[admit - 1] + order[admit]) - order[K - 1]
        mask = _mask_of(m for m in range(M) if arrival[m] <= order[K - 1] + grace)
        tokens = np.maximum(np.rint(rng.lognormal(mean=12.0, sigma=0.5, size=(len(sizes), M))),
                            1).astype(np.uint64)
        return Workload(name, M=M, K=K, learner_dtype="bf16", fragment_sizes=sizes,
                        tokens=tokens, masks=[mask] * len(sizes), seed=2, arrival_s=arrival,
                        grace_s=float(grace), notes="grace window admits 13 of 16")
    if name == "moe4b":
        rng = np.random.default_rng(3)
        sizes = moe_fragments(16, 2048, 1408, 32, 32000)
        M = 16
        tokens = rng.integers(50_000, 500_001, size=(len(sizes), M)).astype(np.uint64)
        masks = []
        for _ in sizes:
            s = int(rng.integers(10, 17))
            masks.append(_mask_of(rng.choice(M, size=s, replace=False)))
        return Workload(name, M=M, K=10, learner_dtype="bf16", fragment_sizes=sizes,
                        tokens=tokens, masks=masks, seed=3,
                        notes="ragged fragments, 10-16 participants each")
    if name == "scale500m":
        rng = np.random.default_rng(4)
        M = 32
        members = rng.choice(M, size=24, replace=False)
        tokens = rng.integers(100_000, 400_001, size=(1, M)).astype(np.uint64)
        return Workload(name, M=M, K=24, learner_dtype="bf16", fragment_sizes=[500_000_000],
                        tokens=tokens, masks=[_mask_of(members)], seed=4, repeats=20,
                        notes="quorum 24 of 32, 20 back-to-back merges")
    raise KeyError(name)


WORKLOADS = ("tiny", "dense150m", "dense1b3", "moe4b", "scale500m")


def scaled(w: Workload, factor: float, align: int = 1) -> Workload:
    """Same structure with every fragment shrunk by ``factor`` (for parity runs
    the oracle can finish); sizes stay ragged (not rounded to a tile)."""
    sizes = [max(1, int(n * factor)) for n in w.fragment_sizes]
    if align > 1:
        sizes = [max(align, n - n % align) for n in sizes]
    return Workload(w.name + f"@{factor:g}", M=w.M, K=w.K, learner_dtype=w.learner_dtype,
                    fragment_sizes=sizes, tokens=w.tokens, masks=w.masks, seed=w.seed,
                    repeats=w.repeats, arrival_s=w.arrival_s, grace_s=w.grace_s, notes=w.notes,
                    steps=w.steps)


# ---- parameter values ---------------------------------------------------------

def fragment_cpu(n: int, M: int, learner_dtype: str, seed: int, *, present=None):
    """Host arrays for one fragment: (theta f32[n], v f32[n] zeros, learners list).

    Learner copies are float32 arrays, or uint16 arrays holding bf16 bits when
    ``learner_dtype == "bf16"``.  ``present`` (iterable of learner ids) limits
    which copies are materialised; the others are ``None``.
    """
    import torch

    g = torch.Generator().manual_seed(int(seed))
    theta = torch.randn(n, generator=g, dtype=torch.float32) * THETA_STD
    learners = []
    keep = None if present is None else set(int(m) for m in present)
    for m in range(M):
        noise = torch.randn(n, generator=g, dtype=torch.float32) * LEARNER_NOISE_STD
        if keep is not None and m not in keep:
            learners.append(None)
            continue
        x = theta + noise
        if learner_dtype == "bf16":
            learners.append(x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy())
        else:
            learners.append(x.numpy().copy())
    return theta.numpy().copy(), np.zeros(n, dtype=np.float32), learners


def fill_fragment_gpu(theta, momentum, learners, seed: int, chunk: int = 1 << 26):
    """Fill device tensors in place with the same recipe, chunk by chunk.

    ``theta``/``momentum``: float32 CUDA tensors of n elements; ``learners``: list
    of CUDA tensors (float32 or bfloat16) or ``None``.  Values differ from
    :func:`fragment_cpu` (another generator); the distribution is the same.
    """
    import torch

    n = theta.numel()
    g = torch.Generator(device=theta.device).manual_seed(int(seed))
    momentum.zero_()
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        base = torch.randn(hi - lo, generator=g, device=theta.device, dtype=torch.float32)
        base.mul_(THETA_STD)
        theta[lo:hi].copy_(base)
        for t in learners:
            if t is None:
                continue
            noise = torch.randn(hi - lo, generator=g, device=theta.device, dtype=torch.float32)
            noise.mul_(LEARNER_NOISE_STD).add_(base)
            t[lo:hi].copy_(noise)


def dense_tensor_list(layers: int, d: int, d_ff: int, vocab: int):
    """(element count, transformer layer or -1) for every tensor of a dense decoder, in
    model order: embedding, per layer q k v o up down and two norm gains, final norm, head."""
    tensors = [(vocab * d, -1)]
    for l in range(layers):
        tensors += [(d * d, l)] * 4 + [(d * d_ff, l)] * 2 + [(d, l)] * 2
    tensors += [(d, -1), (vocab * d, -1)]
    return tensors


# ---- event tapes ------------------------------------------------------------------

def synthetic_tape(M: int, P: int, H: int, offsets, steps_total: int, seed: int, *,
                   batch_tokens: int = 4096, fail_prob: float = 0.08, recover_prob: float = 0.4,
                   straggle_prob: float = 0.15):
    """A seeded stand-in for a recorded event tape: per syncer step, the arrival time
    of every learner's report (inf while the learner is down) and the per-(fragment,
    learner) token / step counters accumulated since that learner last received the
    fragment.  A learner that is up takes one inner step per syncer step (none when it
    straggles); counters of a fragment are reset for every learner that is up when the
    fragment is due (it then receives the new global fragment).
    Returns a list of dicts {arrival_s, tokens, steps} (plain lists).
    """
    rng = np.random.default_rng(seed)
    up = [True] * M
    tokens = np.zeros((P, M), dtype=np.int64)
    steps = np.zeros((P, M), dtype=np.int64)
    tape = []
    for t in range(steps_total):
        arrival = []
        for m in range(M):
            if up[m] and rng.random() < fail_prob:
                up[m] = False
            elif not up[m] and rng.random() < recover_prob:
                up[m] = True
            if up[m]:
                took = 0 if rng.random() < straggle_prob else 1
                tokens[:, m] += took * batch_tokens * int(rng.integers(1, 3))
                steps[:, m] += took
                arrival.append(float(np.round(rng.lognormal(0.0, 0.5), 3)))
            else:
                arrival.append(float("inf"))
        tape.append(dict(arrival_s=arrival, tokens=tokens.tolist(), steps=steps.tolist()))
        for p in range(P):
            if t % H == offsets[p]:
                for m in range(M):
                    if up[m]:
                        tokens[p, m] = 0
                        steps[p, m] = 0
    return tape
