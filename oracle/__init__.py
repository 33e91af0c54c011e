"""CPU oracle for the per-fragment merge (TEST INFRASTRUCTURE ONLY).

Thin ctypes wrapper around ``dd_oracle.c`` (plain C99, fp64, single thread).
It is imported by the test-suite, by the smoke check and by the benchmark's
cpu_baseline / reference legs -- never by the product package, and it imports
nothing from it.  bf16 arrays are carried as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dd_oracle.c")
_LIB = os.path.join(_HERE, "libdd_oracle.so")

MAX_LEARNERS = 64
STATUS_OK, STATUS_QUORUM_NOT_MET, STATUS_ZERO_WEIGHT, INVALID = 0, 1, 2, -1
MERGE_AVG, MERGE_RDA = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2``, no OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-Wall", "-Wextra",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Record(ctypes.Structure):
    _fields_ = [
        ("status", ctypes.c_int32),
        ("n_part", ctypes.c_int32),
        ("idx", ctypes.c_uint8 * MAX_LEARNERS),
        ("w_hat", ctypes.c_double * MAX_LEARNERS),
        ("w_total", ctypes.c_double),
        ("delta_sq", ctypes.c_double),
        ("theta_sq", ctypes.c_double),
        ("mom_sq", ctypes.c_double),
        ("delta_m_sq", ctypes.c_double * MAX_LEARNERS),
    ]


@dataclass
class Record:
    status: int
    n_part: int
    idx: list = field(default_factory=list)
    w_hat: list = field(default_factory=list)
    w_total: float = 0.0
    delta_sq: float = 0.0
    theta_sq: float = 0.0
    mom_sq: float = 0.0
    delta_m_sq: list = field(default_factory=list)


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64p = ctypes.POINTER(ctypes.c_uint64)
        lib.ddo_bf16_rne.restype = ctypes.c_uint16
        lib.ddo_bf16_rne.argtypes = [ctypes.c_float]
        lib.ddo_bf16_rne_array.restype = None
        lib.ddo_bf16_rne_array.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t]
        lib.ddo_bf16_to_f32.restype = ctypes.c_float
        lib.ddo_bf16_to_f32.argtypes = [ctypes.c_uint16]
        lib.ddo_participants.restype = ctypes.c_int
        lib.ddo_participants.argtypes = [ctypes.c_uint64, u64p, ctypes.c_int, ctypes.c_int,
                                         ctypes.POINTER(ctypes.c_uint8),
                                         ctypes.POINTER(ctypes.c_int32)]
        lib.ddo_weights.restype = ctypes.c_int
        lib.ddo_weights.argtypes = [u64p, u64p, ctypes.POINTER(ctypes.c_uint8), ctypes.c_int,
                                    ctypes.POINTER(ctypes.c_double),
                                    ctypes.POINTER(ctypes.c_double)]
        lib.ddo_merge_fragment.restype = ctypes.c_int
        lib.ddo_merge_fragment.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_int,
            ctypes.c_int, u64p, u64p, ctypes.c_uint64, ctypes.c_int, ctypes.c_float,
            ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p,
            ctypes.POINTER(_Record)]
        lib.ddo_merge_fragment_rda_stage.restype = ctypes.c_int
        lib.ddo_merge_fragment_rda_stage.argtypes = [
            ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_int,
            ctypes.c_int, u64p, u64p, ctypes.c_uint64, ctypes.c_int, ctypes.c_float, ctypes.c_float,
            ctypes.c_int, ctypes.c_size_t, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
            ctypes.c_void_p, ctypes.POINTER(_Record)]
        lib.ddo_apply_to_learner.restype = None
        lib.ddo_apply_to_learner.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                             ctypes.c_float, ctypes.c_size_t]
        lib.ddo_quantize_int4.restype = None
        lib.ddo_quantize_int4.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                          ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
        lib.ddo_merge_fragment_int4.restype = ctypes.c_int
        lib.ddo_merge_fragment_int4.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p),
            ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, u64p, u64p, ctypes.c_uint64, ctypes.c_int,
            ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p,
            ctypes.POINTER(_Record)]
        lib.ddo_grace_window.restype = ctypes.c_double
        lib.ddo_grace_window.argtypes = [ctypes.c_double] * 5
        lib.ddo_select_quorum.restype = ctypes.c_int
        lib.ddo_select_quorum.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.c_int,
                                          ctypes.c_int, ctypes.c_double,
                                          ctypes.POINTER(ctypes.c_uint64),
                                          ctypes.POINTER(ctypes.c_int32)]
        _lib = lib
    return _lib


def _u64(values):
    arr = (ctypes.c_uint64 * len(values))(*[int(x) for x in values])
    return arr


def bf16_rne(x) -> np.ndarray:
    """fp32 array -> bf16 bit patterns (uint16), round-to-nearest-even."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib.ddo_bf16_rne_array(x.ctypes.data, out.ctypes.data, x.size)
    return out


def bf16_to_f32(h) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32 (exact)."""
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32)


def participants(mask: int, tokens, K: int):
    """Returns (status, idx list)."""
    lib = _load()
    M = len(tokens)
    idx = (ctypes.c_uint8 * MAX_LEARNERS)()
    n_part = ctypes.c_int32(0)
    st = lib.ddo_participants(ctypes.c_uint64(mask & (2**64 - 1)), _u64(tokens), M, K, idx,
                              ctypes.byref(n_part))
    if st == INVALID:
        raise ValueError("oracle: invalid participation arguments")
    return st, [int(idx[j]) for j in range(n_part.value)]


def weights(tokens, steps, idx):
    """Returns (status, w_hat list aligned with idx, w_total)."""
    lib = _load()
    s = len(idx)
    idx_c = (ctypes.c_uint8 * MAX_LEARNERS)(*idx)
    w_hat = (ctypes.c_double * MAX_LEARNERS)()
    W = ctypes.c_double(0.0)
    st = lib.ddo_weights(_u64(tokens), None if steps is None else _u64(steps), idx_c, s, w_hat,
                         ctypes.byref(W))
    if st == INVALID:
        raise ValueError("oracle: tokens > 0 with steps == 0, or token sum beyond 64 bits")
    return st, [float(w_hat[j]) for j in range(s)], float(W.value)


def merge_fragment(theta: np.ndarray, v: np.ndarray, learners, tokens, mask: int, K: int,
                   eta: float, mu: float, *, steps=None, nesterov: bool = True,
                   merge: int = MERGE_AVG, out_bf16: np.ndarray | None = None) -> Record:
    """One syncer update of one fragment, IN PLACE on ``theta`` and ``v``.

    ``theta``/``v``: contiguous float32 arrays of n elements.  ``learners``: list
    of M arrays (all float32, or all uint16 holding bf16 bits) or ``None`` for a
    learner whose copy is not available.  ``out_bf16``: optional uint16[n].
    """
    lib = _load()
    assert theta.dtype == np.float32 and v.dtype == np.float32
    assert theta.flags.c_contiguous and v.flags.c_contiguous and theta.shape == v.shape
    n = theta.size
    M = len(learners)
    present = [a for a in learners if a is not None]
    is_bf16 = bool(present) and present[0].dtype == np.uint16
    ptrs = (ctypes.c_void_p * M)()
    for m, a in enumerate(learners):
        if a is None:
            ptrs[m] = None
            continue
        assert a.dtype == (np.uint16 if is_bf16 else np.float32), "mixed learner dtypes"
        assert a.flags.c_contiguous and a.size == n
        ptrs[m] = a.ctypes.data
    if out_bf16 is not None:
        assert out_bf16.dtype == np.uint16 and out_bf16.size == n and out_bf16.flags.c_contiguous
    rec = _Record()
    rc = lib.ddo_merge_fragment(
        theta.ctypes.data, v.ctypes.data, ptrs, M, int(is_bf16), _u64(tokens),
        None if steps is None else _u64(steps), ctypes.c_uint64(mask & (2**64 - 1)), K,
        ctypes.c_float(eta), ctypes.c_float(mu), int(nesterov), int(merge), n,
        None if out_bf16 is None else out_bf16.ctypes.data, ctypes.byref(rec))
    if rc != 0:
        raise ValueError("oracle: invalid merge arguments")
    s = rec.n_part
    return Record(status=rec.status, n_part=s, idx=[int(rec.idx[j]) for j in range(s)],
                  w_hat=[float(rec.w_hat[j]) for j in range(s)], w_total=float(rec.w_total),
                  delta_sq=float(rec.delta_sq), theta_sq=float(rec.theta_sq),
                  mom_sq=float(rec.mom_sq),
                  delta_m_sq=[float(rec.delta_m_sq[j]) for j in range(s)])


def grace_window(tau, xi_step, xi_quorum, xi_sync, gamma) -> float:
    return float(_load().ddo_grace_window(tau, xi_step, xi_quorum, xi_sync, gamma))


def select_quorum(arrival, K: int, grace: float):
    """Returns (status, mask, n_admitted)."""
    lib = _load()
    M = len(arrival)
    arr = (ctypes.c_double * M)(*[float(a) for a in arrival])
    mask = ctypes.c_uint64(0)
    n_adm = ctypes.c_int32(0)
    st = lib.ddo_select_quorum(arr, M, K, float(grace), ctypes.byref(mask), ctypes.byref(n_adm))
    if st == INVALID:
        raise ValueError("oracle: invalid quorum arguments")
    return st, int(mask.value), int(n_adm.value)


def merge_fragment_rda_stage(stage: int, theta: np.ndarray, v: np.ndarray, learners, tokens, mask: int,
                             K: int, eta: float, mu: float, *, norms_sq=None, dir_sq: float = 0.0,
                             steps=None, nesterov: bool = True, out_bf16: np.ndarray | None = None):
    """One stage (0 norms, 1 direction, 2 outer step) of the radial-directional merge on ONE element
    range of a sharded fragment; the caller sums each stage's output over the ranges before the next
    stage.  ``norms_sq``: the summed stage-0 output (participant order); ``dir_sq``: the summed
    stage-1 output.  Stage 2 updates ``theta`` and ``v`` in place.  Returns (Record, dir_sq of this
    range for stage 1)."""
    lib = _load()
    assert theta.dtype == np.float32 and v.dtype == np.float32 and theta.shape == v.shape
    n, M = theta.size, len(learners)
    present = [a for a in learners if a is not None]
    is_bf16 = bool(present) and present[0].dtype == np.uint16
    ptrs = (ctypes.c_void_p * M)(*[None if a is None else a.ctypes.data for a in learners])
    for a in present:
        assert a.flags.c_contiguous and a.size == n
    norms = None if norms_sq is None else (ctypes.c_double * MAX_LEARNERS)(*[float(x) for x in norms_sq])
    dsq = ctypes.c_double(float(dir_sq))
    rec = _Record()
    rc = lib.ddo_merge_fragment_rda_stage(
        int(stage), theta.ctypes.data, v.ctypes.data, ptrs, M, int(is_bf16), _u64(tokens),
        None if steps is None else _u64(steps), ctypes.c_uint64(mask & (2**64 - 1)), K, ctypes.c_float(eta),
        ctypes.c_float(mu), int(nesterov), n, norms, ctypes.byref(dsq),
        None if out_bf16 is None else out_bf16.ctypes.data, ctypes.byref(rec))
    if rc != 0:
        raise ValueError("oracle: invalid arguments of a radial-directional stage")
    s = rec.n_part
    out = Record(status=rec.status, n_part=s, idx=[int(rec.idx[j]) for j in range(s)],
                 w_hat=[float(rec.w_hat[j]) for j in range(s)], w_total=float(rec.w_total),
                 delta_sq=float(rec.delta_sq), theta_sq=float(rec.theta_sq), mom_sq=float(rec.mom_sq),
                 delta_m_sq=[float(rec.delta_m_sq[j]) for j in range(s)])
    return out, float(dsq.value)


def apply_to_learner(learner: np.ndarray, theta: np.ndarray, alpha: float) -> None:
    """theta_m <- alpha theta_m + (1 - alpha) Theta, IN PLACE on ``learner`` (float32 or
    uint16 holding bf16 bits)."""
    lib = _load()
    assert theta.dtype == np.float32 and learner.size == theta.size
    assert learner.flags.c_contiguous and theta.flags.c_contiguous
    lib.ddo_apply_to_learner(learner.ctypes.data, int(learner.dtype == np.uint16), theta.ctypes.data,
                             ctypes.c_float(alpha), theta.size)


def grace_controller_window(tau, gamma, beta, observations) -> float:
    """Moving averages x <- beta x + (1 - beta) obs (first observation initialises),
    then the largest admissible grace window; written out with plain floats."""
    xs = None
    for obs in observations:
        xs = list(obs) if xs is None else [beta * x + (1.0 - beta) * o for x, o in zip(xs, obs)]
    if xs is None:
        return 0.0
    return grace_window(tau, xs[0], xs[1], xs[2], gamma)


INT4_BLOCK = 128


def quantize_int4(theta: np.ndarray, learner: np.ndarray):
    """Outer gradient Theta - theta of one learner as int4 codes + one float32 scale per
    128 elements.  Returns (codes uint8[ceil(n/2)], scales float32[ceil(n/128)])."""
    lib = _load()
    n = theta.size
    assert theta.dtype == np.float32 and learner.size == n
    codes = np.zeros((n + 1) // 2, dtype=np.uint8)
    scales = np.zeros((n + INT4_BLOCK - 1) // INT4_BLOCK, dtype=np.float32)
    lib.ddo_quantize_int4(theta.ctypes.data, learner.ctypes.data, int(learner.dtype == np.uint16), n,
                          codes.ctypes.data, scales.ctypes.data)
    return codes, scales


def dequantize_int4(codes: np.ndarray, scales: np.ndarray, n: int) -> np.ndarray:
    """(code - 8) * scale in float32, for tests."""
    i = np.arange(n)
    nib = (codes[i // 2] >> (4 * (i & 1))) & 15
    return ((nib.astype(np.int32) - 8).astype(np.float32) * scales[i // INT4_BLOCK]).astype(np.float32)


def merge_fragment_int4(theta: np.ndarray, v: np.ndarray, codes, scales, tokens, mask: int, K: int,
                        eta: float, mu: float, *, steps=None, nesterov: bool = True,
                        out_bf16: np.ndarray | None = None) -> Record:
    """The merge with int4-compressed outer gradients, IN PLACE on theta and v."""
    lib = _load()
    M = len(codes)
    n = theta.size
    cp = (ctypes.c_void_p * M)(*[None if a is None else a.ctypes.data for a in codes])
    sp = (ctypes.c_void_p * M)(*[None if a is None else a.ctypes.data for a in scales])
    rec = _Record()
    rc = lib.ddo_merge_fragment_int4(
        theta.ctypes.data, v.ctypes.data, cp, sp, M, _u64(tokens),
        None if steps is None else _u64(steps), ctypes.c_uint64(mask & (2**64 - 1)), K,
        ctypes.c_float(eta), ctypes.c_float(mu), int(nesterov), n,
        None if out_bf16 is None else out_bf16.ctypes.data, ctypes.byref(rec))
    if rc != 0:
        raise ValueError("oracle: invalid int4 merge arguments")
    s = rec.n_part
    return Record(status=rec.status, n_part=s, idx=[int(rec.idx[j]) for j in range(s)],
                  w_hat=[float(rec.w_hat[j]) for j in range(s)], w_total=float(rec.w_total),
                  delta_sq=float(rec.delta_sq), theta_sq=float(rec.theta_sq),
                  mom_sq=float(rec.mom_sq), delta_m_sq=[0.0] * s)


# ---- all-cores CPU baseline (benchmark only; not the checked oracle) ---------------------

_PAR_SRC = os.path.join(_HERE, "dd_cpu_parallel.c")
_PAR_LIB = os.path.join(_HERE, "libdd_cpu_parallel.so")
_par = None


def build_parallel(force: bool = False) -> str:
    if force or not os.path.exists(_PAR_LIB) or os.path.getmtime(_PAR_LIB) < os.path.getmtime(_PAR_SRC):
        tmp = _PAR_LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall",
                               "-ffp-contract=off", "-o", tmp, _PAR_SRC])
        os.replace(tmp, _PAR_LIB)
    return _PAR_LIB


def merge_fragment_all_cores(theta, v, learners, tokens, mask, K, eta, mu, *, nesterov=True):
    """The direct-averaging merge with the element loop spread over all host cores
    (OpenMP).  Participation and weights come from the single-threaded oracle.
    Returns ||Delta||^2, or None when the quorum is not met."""
    global _par
    if _par is None:
        _par = ctypes.CDLL(build_parallel())
        _par.ddp_merge_fragment.restype = ctypes.c_double
        _par.ddp_merge_fragment.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p),
            ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.c_int, ctypes.c_float,
            ctypes.c_float, ctypes.c_int, ctypes.c_size_t]
    st, idx = participants(mask, tokens, K)
    if st != STATUS_OK:
        return None
    _, w_hat, _ = weights(tokens, None, idx)
    chosen = [learners[m] for m in idx]
    is_bf16 = chosen[0].dtype == np.uint16
    ptrs = (ctypes.c_void_p * len(idx))(*[a.ctypes.data for a in chosen])
    wh = (ctypes.c_double * len(idx))(*w_hat)
    return float(_par.ddp_merge_fragment(theta.ctypes.data, v.ctypes.data, ptrs, wh, len(idx),
                                         int(is_bf16), ctypes.c_float(eta), ctypes.c_float(mu),
                                         int(nesterov), theta.size))
