"""ctypes binding of libddmerge (argument marshalling only).

Every step of the merge runs in the CUDA library; this module turns torch
tensors into raw device pointers, host lists into C arrays, and the device-side
``dd_merge_record`` back into Python values.  There is no CPU fallback: if the
library is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

MAX_LEARNERS = 64
F32, BF16 = 0, 1
OK = 0
ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_ALIAS, ERR_TOO_MANY_LEARNERS, ERR_CUDA, ERR_TOO_LARGE = \
    -1, -2, -3, -4, -5, -6
STATUS_OK, STATUS_QUORUM_NOT_MET, STATUS_ZERO_WEIGHT, STATUS_WAIT_LIMIT = 0, 1, 2, 3
HEAVY_BALL, DIAG_PER_LEARNER, DIAG_STATE, RDA_THREE_PASS = 1, 2, 4, 8
DEBUG_EXPIRE_WAIT = 1 << 30
MERGE_AVG, MERGE_RDA = 0, 1
RDA_PASS_NORMS, RDA_PASS_DIRECTION, RDA_PASS_APPLY = 0, 1, 2
FRAG_LAYER, FRAG_TENSOR, FRAG_BALANCED = 0, 1, 2

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libddmerge.so")

EXPORTS = (
    "dd_create", "dd_destroy", "dd_merge_fragment", "dd_merge_fragments_batched",
    "dd_merge_fragment_push", "dd_merge_fragments_batched_push", "dd_merge_fragments_batched_rda_push", "dd_merge_fragments_batched_rda_pass",
    "dd_merge_fragment_host", "dd_merge_fragments_batched_host", "dd_merge_fragment_int4_host",
    "dd_merge_fragments_batched_noalloc",
    "dd_merge_fragment_rda", "dd_merge_fragments_batched_rda",
    "dd_quantize_outer_gradient_int4", "dd_merge_fragment_int4",
    "dd_broadcast_fragment", "dd_grace_controller_init", "dd_grace_controller_observe",
    "dd_grace_controller_window", "dd_plan_fragments", "dd_select_quorum", "dd_grace_window", "dd_status_string", "dd_last_cuda_error",
    "dd_launch_geometry", "dd_launch_shape",
)


class CRecord(ctypes.Structure):
    """Mirror of ``dd_merge_record``."""
    _fields_ = [
        ("status", ctypes.c_int32),
        ("n_part", ctypes.c_int32),
        ("idx", ctypes.c_uint8 * MAX_LEARNERS),
        ("w_hat", ctypes.c_float * MAX_LEARNERS),
        ("w_total", ctypes.c_double),
        ("delta_sq", ctypes.c_double),
        ("theta_sq", ctypes.c_double),
        ("mom_sq", ctypes.c_double),
        ("delta_m_sq", ctypes.c_double * MAX_LEARNERS),
    ]


class CFragmentDesc(ctypes.Structure):
    """Mirror of ``dd_fragment_desc``."""
    _fields_ = [
        ("global_", ctypes.c_void_p),
        ("momentum", ctypes.c_void_p),
        ("out_bf16", ctypes.c_void_p),
        ("learner_ptrs", ctypes.POINTER(ctypes.c_void_p)),
        ("tokens", ctypes.POINTER(ctypes.c_uint64)),
        ("steps", ctypes.POINTER(ctypes.c_uint64)),
        ("quorum_mask", ctypes.c_uint64),
        ("K", ctypes.c_int32),
        ("n", ctypes.c_uint64),
    ]


class CGraceController(ctypes.Structure):
    """Mirror of ``dd_grace_controller``."""
    _fields_ = [("tau", ctypes.c_double), ("gamma", ctypes.c_double), ("beta", ctypes.c_double),
                ("xi_step", ctypes.c_double), ("xi_quorum", ctypes.c_double),
                ("xi_sync", ctypes.c_double), ("n_obs", ctypes.c_int32)]


RECORD_BYTES = ctypes.sizeof(CRecord)


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2604_21428_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, u64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint64)
    lib.dd_create.restype = ctypes.c_int
    lib.dd_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
    lib.dd_destroy.restype = ctypes.c_int
    lib.dd_destroy.argtypes = [vp]
    lib.dd_merge_fragment.restype = ctypes.c_int
    lib.dd_merge_fragment.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, vp, vp, vp]
    lib.dd_merge_fragments_batched.restype = ctypes.c_int
    lib.dd_merge_fragments_batched.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_float, ctypes.c_float, ctypes.c_uint32, vp, vp]
    lib.dd_merge_fragment_push.restype = ctypes.c_int
    lib.dd_merge_fragment_push.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, ctypes.c_uint64,
        vp, vp, vp]
    lib.dd_merge_fragments_batched_push.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_push.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), u64p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_float, ctypes.c_float, ctypes.c_uint32, vp, vp]
    lib.dd_merge_fragment_rda.restype = ctypes.c_int
    lib.dd_merge_fragment_rda.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, vp, vp, vp, vp]
    lib.dd_merge_fragments_batched_rda.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_rda.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint8), vp, vp,
        ctypes.c_size_t, vp]
    lib.dd_merge_fragments_batched_rda_push.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_rda_push.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), u64p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint8), vp, vp,
        ctypes.c_size_t, vp]
    lib.dd_merge_fragments_batched_rda_pass.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_rda_pass.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), u64p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
        ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint8), vp, vp,
        ctypes.c_size_t, ctypes.c_int, vp]
    lib.dd_quantize_outer_gradient_int4.restype = ctypes.c_int
    lib.dd_quantize_outer_gradient_int4.argtypes = [vp, vp, vp, ctypes.c_int, ctypes.c_size_t, vp, vp, vp]
    lib.dd_merge_fragment_int4.restype = ctypes.c_int
    lib.dd_merge_fragment_int4.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, vp, vp, vp]
    lib.dd_merge_fragment_host.restype = ctypes.c_int
    lib.dd_merge_fragment_host.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, vp,
        ctypes.POINTER(CRecord), ctypes.c_size_t, vp]
    lib.dd_merge_fragments_batched_host.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_host.argtypes = [
        vp, ctypes.POINTER(CFragmentDesc), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float,
        ctypes.c_float, ctypes.c_uint32, ctypes.POINTER(CRecord), ctypes.c_size_t, vp]
    lib.dd_merge_fragment_int4_host.restype = ctypes.c_int
    lib.dd_merge_fragment_int4_host.argtypes = [
        vp, vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, u64p, u64p, ctypes.c_uint64,
        ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, ctypes.c_size_t, vp,
        ctypes.POINTER(CRecord), ctypes.c_size_t, vp]
    lib.dd_merge_fragments_batched_noalloc.restype = ctypes.c_int
    lib.dd_merge_fragments_batched_noalloc.argtypes = [
        ctypes.POINTER(CFragmentDesc), ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float,
        ctypes.c_float, ctypes.c_uint32, vp, vp]
    lib.dd_select_quorum.restype = ctypes.c_int
    lib.dd_select_quorum.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.c_int,
                                     ctypes.c_double, u64p, ctypes.POINTER(ctypes.c_int)]
    lib.dd_broadcast_fragment.restype = ctypes.c_int
    lib.dd_broadcast_fragment.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.c_int, ctypes.c_int,
                                          ctypes.c_uint64, ctypes.c_float, ctypes.c_size_t, vp]
    gcp = ctypes.POINTER(CGraceController)
    lib.dd_grace_controller_init.restype = ctypes.c_int
    lib.dd_grace_controller_init.argtypes = [gcp, ctypes.c_double, ctypes.c_double, ctypes.c_double]
    lib.dd_grace_controller_observe.restype = ctypes.c_int
    lib.dd_grace_controller_observe.argtypes = [gcp, ctypes.c_double, ctypes.c_double, ctypes.c_double]
    lib.dd_grace_controller_window.restype = ctypes.c_double
    lib.dd_grace_controller_window.argtypes = [gcp]
    lib.dd_plan_fragments.restype = ctypes.c_int
    lib.dd_plan_fragments.argtypes = [u64p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int32),
                                      u64p]
    lib.dd_grace_window.restype = ctypes.c_double
    lib.dd_grace_window.argtypes = [ctypes.c_double] * 5
    lib.dd_status_string.restype = ctypes.c_char_p
    lib.dd_status_string.argtypes = [ctypes.c_int]
    lib.dd_last_cuda_error.restype = ctypes.c_char_p
    lib.dd_last_cuda_error.argtypes = [vp]
    lib.dd_launch_geometry.restype = ctypes.c_int
    lib.dd_launch_geometry.argtypes = [vp, ctypes.c_int] + [ctypes.POINTER(ctypes.c_int)] * 3
    lib.dd_launch_shape.restype = ctypes.c_int
    lib.dd_launch_shape.argtypes = [ctypes.c_int] * 4 + [ctypes.POINTER(ctypes.c_int)] * 2
    return lib


lib = _load()


class DDMergeError(RuntimeError):
    def __init__(self, rc: int, detail: str = ""):
        self.rc = rc
        msg = lib.dd_status_string(rc).decode()
        super().__init__(f"libddmerge: {msg} (rc={rc})" + (f": {detail}" if detail else ""))


@dataclass
class Record:
    status: int
    n_part: int
    idx: list = field(default_factory=list)
    w_hat: list = field(default_factory=list)      # float32 values
    w_total: float = 0.0
    delta_sq: float = 0.0
    theta_sq: float = 0.0
    mom_sq: float = 0.0
    delta_m_sq: list = field(default_factory=list)


def _ptr(x) -> int | None:
    """Device/host address of a tensor-like, or the integer itself."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return int(x.data_ptr())


def _u64_array(values):
    if isinstance(values, ctypes.Array):
        return values
    return (ctypes.c_uint64 * len(values))(*[int(v) for v in values])


def pack_pointers(tensors):
    """The addresses of ``tensors`` (tensors / ints / None) as a C array.  Every entry point that
    takes a list of learner buffers also takes this array, which saves the per-call marshalling
    when the same buffers are merged again and again (pass ``learner_dtype`` explicitly then)."""
    return (ctypes.c_void_p * len(tensors))(*[_ptr(t) for t in tensors])


def pack_u64(values):
    """Token or step counts as a C array of uint64 (accepted wherever a list of counts is)."""
    return (ctypes.c_uint64 * len(values))(*[int(v) for v in values])


def _pointer_array(learners):
    return learners if isinstance(learners, ctypes.Array) else pack_pointers(learners)


def _stream_handle(stream) -> int | None:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def record_field_columns(name: str):
    """(first, last + 1) float64 columns of ``dd_merge_record`` field ``name`` in a records buffer
    viewed as float64 [count, RECORD_BYTES // 8] -- for summing fields across GPUs in place."""
    f = getattr(CRecord, name)
    assert f.offset % 8 == 0 and f.size % 8 == 0, name
    return f.offset // 8, (f.offset + f.size) // 8


def new_records(count: int, device=None):
    """Device buffer for ``count`` records (a uint8 torch tensor)."""
    import torch
    return torch.zeros(count * RECORD_BYTES, dtype=torch.uint8, device=device or "cuda")


def read_records(buf, count: int | None = None) -> list:
    """Copies the record buffer to the host (synchronises) and parses it."""
    raw = bytes(buf.cpu().numpy().tobytes())
    count = len(raw) // RECORD_BYTES if count is None else count
    return [_parse_record(CRecord.from_buffer_copy(raw, p * RECORD_BYTES)) for p in range(count)]


def _parse_record(r: CRecord) -> Record:
    s = max(0, min(int(r.n_part), MAX_LEARNERS))
    return Record(status=int(r.status), n_part=int(r.n_part),
                  idx=[int(r.idx[j]) for j in range(s)],
                  w_hat=[float(r.w_hat[j]) for j in range(s)],
                  w_total=float(r.w_total), delta_sq=float(r.delta_sq),
                  theta_sq=float(r.theta_sq), mom_sq=float(r.mom_sq),
                  delta_m_sq=[float(r.delta_m_sq[j]) for j in range(s)])


class Context:
    """Owns a ``dd_ctx`` (GPU binding + diagnostics workspace)."""

    def __init__(self, device: int = -1):
        handle = ctypes.c_void_p()
        rc = lib.dd_create(ctypes.byref(handle), int(device))
        if rc != OK:
            raise DDMergeError(rc, "dd_create")
        self._h = handle

    def close(self):
        if getattr(self, "_h", None):
            lib.dd_destroy(self._h)
            self._h = None

    def __del__(self):  # best effort
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            detail = lib.dd_last_cuda_error(self._h).decode() if rc == ERR_CUDA else ""
            raise DDMergeError(rc, detail)

    def launch_geometry(self, dtype: int = BF16):
        g, b, t = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        self._check(lib.dd_launch_geometry(self._h, dtype, ctypes.byref(g), ctypes.byref(b),
                                           ctypes.byref(t)))
        return g.value, b.value, t.value

    def merge_fragment(self, global_, momentum, learners, tokens, quorum_mask: int, K: int,
                       outer_lr: float, outer_mu: float, *, n: int | None = None,
                       learner_dtype: int | None = None, steps=None, flags: int = 0,
                       out_bf16=None, record=None, stream=None) -> None:
        """``dd_merge_fragment``: ``learners`` is a list of tensors / addresses / None."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        ptrs = _pointer_array(learners)
        self._check(lib.dd_merge_fragment(
            self._h, _ptr(global_), _ptr(momentum), ptrs, M, learner_dtype, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n), _ptr(out_bf16),
            _ptr(record), _stream_handle(stream)))

    def prepare_merge_fragment(self, global_, momentum, learners, tokens, K: int, outer_lr: float,
                               outer_mu: float, *, n: int | None = None, learner_dtype: int | None = None,
                               steps=None, flags: int = 0, out_bf16=None, record=None, stream=None):
        """``dd_merge_fragment`` with every argument but the quorum mask marshalled once: returns
        ``call(quorum_mask)``.  For a syncer that merges the same buffers step after step the
        per-call cost is then the C call alone.  ``tokens`` (and ``steps``) may be ``pack_u64``
        arrays that the caller updates in place between calls; the tensors must stay alive."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        fixed_head = (self._h, _ptr(global_), _ptr(momentum), _pointer_array(learners), M, learner_dtype,
                      _u64_array(tokens), None if steps is None else _u64_array(steps))
        fixed_tail = (int(K), ctypes.c_float(outer_lr), ctypes.c_float(outer_mu), ctypes.c_uint32(flags),
                      ctypes.c_size_t(n), _ptr(out_bf16), _ptr(record), _stream_handle(stream))
        fn, check = lib.dd_merge_fragment, self._check

        def call(quorum_mask: int) -> None:
            rc = fn(*fixed_head, quorum_mask & 0xFFFFFFFFFFFFFFFF, *fixed_tail)
            if rc != OK:
                check(rc)
        return call

    def merge_fragment_push(self, global_, momentum, learners, tokens, quorum_mask: int, K: int,
                            outer_lr: float, outer_mu: float, push_mask: int, *, n: int | None = None,
                            learner_dtype: int | None = None, steps=None, flags: int = 0,
                            out_bf16=None, record=None, stream=None) -> None:
        """``dd_merge_fragment_push``: the merge, and Theta' written over the copies of the
        learners in ``push_mask`` in the same pass."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        ptrs = _pointer_array(learners)
        self._check(lib.dd_merge_fragment_push(
            self._h, _ptr(global_), _ptr(momentum), ptrs, M, learner_dtype, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n),
            ctypes.c_uint64(push_mask & (2**64 - 1)), _ptr(out_bf16), _ptr(record),
            _stream_handle(stream)))

    def merge_fragments_batched_push(self, fragments, push_masks, M: int, learner_dtype: int,
                                     outer_lr: float, outer_mu: float, *, flags: int = 0, records=None,
                                     stream=None) -> None:
        """``dd_merge_fragments_batched_push``: ``push_masks`` holds one mask per fragment."""
        P = len(fragments)
        descs, _keep = _pack_descs(fragments, M)
        self._check(lib.dd_merge_fragments_batched_push(
            self._h, descs, _u64_array([int(x) & (2**64 - 1) for x in push_masks]), P, M, learner_dtype,
            ctypes.c_float(outer_lr), ctypes.c_float(outer_mu), ctypes.c_uint32(flags), _ptr(records),
            _stream_handle(stream)))

    def merge_fragment_rda(self, global_, momentum, learners, tokens, quorum_mask: int, K: int,
                           outer_lr: float, outer_mu: float, *, n: int | None = None,
                           learner_dtype: int | None = None, steps=None, flags: int = 0,
                           out_bf16=None, record=None, scratch=None, stream=None) -> None:
        """``dd_merge_fragment_rda``: radial-directional merge of one fragment."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        ptrs = _pointer_array(learners)
        self._check(lib.dd_merge_fragment_rda(
            self._h, _ptr(global_), _ptr(momentum), ptrs, M, learner_dtype, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n), _ptr(out_bf16),
            _ptr(record), _ptr(scratch), _stream_handle(stream)))

    def merge_fragments_batched_rda(self, fragments, M: int, learner_dtype: int, outer_lr: float,
                                    outer_mu: float, *, merge_kinds=None, flags: int = 0,
                                    records=None, scratch=None, stream=None, push_masks=None) -> None:
        """``dd_merge_fragments_batched_rda``: ``merge_kinds`` is a list of MERGE_AVG /
        MERGE_RDA per fragment (None = all RDA); ``scratch`` an optional float32 tensor.
        With ``push_masks`` (one mask per fragment): ``dd_merge_fragments_batched_rda_push``."""
        P = len(fragments)
        descs, _keep = _pack_descs(fragments, M)
        kinds = None if merge_kinds is None else (ctypes.c_uint8 * P)(*[int(k) for k in merge_kinds])
        tail = (ctypes.c_uint32(flags), kinds, _ptr(records), _ptr(scratch),
                ctypes.c_size_t(0 if scratch is None else int(scratch.numel())), _stream_handle(stream))
        if push_masks is None:
            self._check(lib.dd_merge_fragments_batched_rda(
                self._h, descs, P, M, learner_dtype, ctypes.c_float(outer_lr), ctypes.c_float(outer_mu),
                *tail))
        else:
            self._check(lib.dd_merge_fragments_batched_rda_push(
                self._h, descs, _u64_array([int(x) & (2**64 - 1) for x in push_masks]), P, M,
                learner_dtype, ctypes.c_float(outer_lr), ctypes.c_float(outer_mu), *tail))


    def merge_fragments_batched_rda_pass(self, fragments, M: int, learner_dtype: int, outer_lr: float,
                                         outer_mu: float, pass_index: int, *, records, scratch,
                                         merge_kinds=None, flags: int = 0, push_masks=None,
                                         stream=None) -> None:
        """``dd_merge_fragments_batched_rda_pass``: one of the three passes (RDA_PASS_NORMS,
        RDA_PASS_DIRECTION, RDA_PASS_APPLY) over this GPU's shard of every fragment; the caller
        sums the hand-over fields of ``records`` across the shards between the passes."""
        P = len(fragments)
        descs, _keep = _pack_descs(fragments, M)
        kinds = None if merge_kinds is None else (ctypes.c_uint8 * P)(*[int(k) for k in merge_kinds])
        pm = None if push_masks is None else _u64_array([int(x) & (2**64 - 1) for x in push_masks])
        self._check(lib.dd_merge_fragments_batched_rda_pass(
            self._h, descs, pm, P, M, learner_dtype, ctypes.c_float(outer_lr), ctypes.c_float(outer_mu),
            ctypes.c_uint32(flags), kinds, _ptr(records), _ptr(scratch),
            ctypes.c_size_t(int(scratch.numel())), int(pass_index), _stream_handle(stream)))
    def broadcast_fragment(self, global_, learners, apply_mask: int, alpha: float = 0.0, *,
                           n: int | None = None, learner_dtype: int | None = None,
                           stream=None) -> None:
        """``dd_broadcast_fragment``: theta_m <- alpha theta_m + (1 - alpha) Theta' for the
        learners selected by ``apply_mask``."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        ptrs = _pointer_array(learners)
        self._check(lib.dd_broadcast_fragment(
            self._h, _ptr(global_), ptrs, M, learner_dtype,
            ctypes.c_uint64(apply_mask & (2**64 - 1)), ctypes.c_float(alpha), ctypes.c_size_t(n),
            _stream_handle(stream)))

    def quantize_outer_gradient_int4(self, global_, learner, codes, scales, *, n: int | None = None,
                                     learner_dtype: int | None = None, stream=None) -> None:
        """``dd_quantize_outer_gradient_int4``: ``codes`` uint8[(n+1)//2], ``scales``
        float32[ceil(n/128)], both device tensors written in place."""
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype([learner])
        self._check(lib.dd_quantize_outer_gradient_int4(
            self._h, _ptr(global_), _ptr(learner), learner_dtype, ctypes.c_size_t(n), _ptr(codes),
            _ptr(scales), _stream_handle(stream)))

    def merge_fragment_int4(self, global_, momentum, codes, scales, tokens, quorum_mask: int, K: int,
                            outer_lr: float, outer_mu: float, *, n: int | None = None, steps=None,
                            flags: int = 0, out_bf16=None, record=None, stream=None) -> None:
        """``dd_merge_fragment_int4``: ``codes`` / ``scales`` are lists of M device tensors
        (or None for absent learners)."""
        M = len(codes)
        if n is None:
            n = int(global_.numel())
        cp = (ctypes.c_void_p * M)(*[_ptr(t) for t in codes])
        sp = (ctypes.c_void_p * M)(*[_ptr(t) for t in scales])
        self._check(lib.dd_merge_fragment_int4(
            self._h, _ptr(global_), _ptr(momentum), cp, sp, M, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n), _ptr(out_bf16),
            _ptr(record), _stream_handle(stream)))

    def merge_fragment_host(self, global_, momentum, learners, tokens, quorum_mask: int, K: int,
                            outer_lr: float, outer_mu: float, *, n: int | None = None,
                            learner_dtype: int | None = None, steps=None, flags: int = 0,
                            out_bf16=None, want_record: bool = True, chunk_elems: int = 0,
                            stream=None):
        """``dd_merge_fragment_host``: all tensors are HOST tensors (ideally pinned).
        Blocks until the results are in host memory; returns the fragment's Record."""
        M = len(learners)
        if n is None:
            n = int(global_.numel())
        if learner_dtype is None:
            learner_dtype = _infer_dtype(learners)
        ptrs = _pointer_array(learners)
        rec = CRecord()
        self._check(lib.dd_merge_fragment_host(
            self._h, _ptr(global_), _ptr(momentum), ptrs, M, learner_dtype, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n), _ptr(out_bf16),
            ctypes.byref(rec) if want_record else None, ctypes.c_size_t(chunk_elems),
            _stream_handle(stream)))
        return _parse_record(rec) if want_record else None

    def merge_fragments_batched_host(self, fragments, M: int, learner_dtype: int, outer_lr: float,
                                     outer_mu: float, *, flags: int = 0, want_records: bool = True,
                                     chunk_elems: int = 0, stream=None):
        """``dd_merge_fragments_batched_host``: like ``merge_fragments_batched`` with every tensor
        of every fragment in HOST memory (ideally pinned).  Blocks until the results are in host
        memory; returns the fragments' Records (or None)."""
        P = len(fragments)
        descs, _keep = _pack_descs(fragments, M)
        recs = (CRecord * max(P, 1))() if want_records else None
        self._check(lib.dd_merge_fragments_batched_host(
            self._h, descs, P, M, learner_dtype, ctypes.c_float(outer_lr), ctypes.c_float(outer_mu),
            ctypes.c_uint32(flags), recs, ctypes.c_size_t(chunk_elems), _stream_handle(stream)))
        return [_parse_record(recs[p]) for p in range(P)] if want_records else None

    def merge_fragment_int4_host(self, global_, momentum, codes, scales, tokens, quorum_mask: int, K: int,
                                 outer_lr: float, outer_mu: float, *, n: int | None = None, steps=None,
                                 flags: int = 0, out_bf16=None, want_record: bool = True,
                                 chunk_elems: int = 0, stream=None):
        """``dd_merge_fragment_int4_host``: ``codes`` / ``scales`` are lists of M HOST tensors (or
        None for absent learners); ``global_`` and ``momentum`` host tensors updated in place.
        Blocks until the results are in host memory; returns the fragment's Record."""
        M = len(codes)
        if n is None:
            n = int(global_.numel())
        cp = (ctypes.c_void_p * M)(*[_ptr(t) for t in codes])
        sp = (ctypes.c_void_p * M)(*[_ptr(t) for t in scales])
        rec = CRecord()
        self._check(lib.dd_merge_fragment_int4_host(
            self._h, _ptr(global_), _ptr(momentum), cp, sp, M, _u64_array(tokens),
            None if steps is None else _u64_array(steps),
            ctypes.c_uint64(quorum_mask & (2**64 - 1)), int(K), ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), ctypes.c_size_t(n), _ptr(out_bf16),
            ctypes.byref(rec) if want_record else None, ctypes.c_size_t(chunk_elems),
            _stream_handle(stream)))
        return _parse_record(rec) if want_record else None

    def merge_fragments_batched(self, fragments, M: int, learner_dtype: int, outer_lr: float,
                                outer_mu: float, *, flags: int = 0, records=None,
                                stream=None) -> None:
        """``dd_merge_fragments_batched``: ``fragments`` is a list of dicts with keys
        global_, momentum, learners, tokens, quorum_mask, K, n and optionally
        steps, out_bf16."""
        P = len(fragments)
        descs, _keep = _pack_descs(fragments, M)
        self._check(lib.dd_merge_fragments_batched(
            self._h, descs, P, M, learner_dtype, ctypes.c_float(outer_lr),
            ctypes.c_float(outer_mu), ctypes.c_uint32(flags), _ptr(records),
            _stream_handle(stream)))


def _pack_descs(fragments, M: int):
    """Host-side ``dd_fragment_desc`` array for a list of fragment dicts."""
    P = len(fragments)
    descs = (CFragmentDesc * max(P, 1))()
    keep = []
    for p, f in enumerate(fragments):
        ptrs = (ctypes.c_void_p * M)(*[_ptr(t) for t in f["learners"]])
        tok = _u64_array(f["tokens"])
        stp = None if f.get("steps") is None else _u64_array(f["steps"])
        keep += [ptrs, tok, stp]
        d = descs[p]
        d.global_ = _ptr(f["global_"])
        d.momentum = _ptr(f["momentum"])
        d.out_bf16 = _ptr(f.get("out_bf16"))
        d.learner_ptrs = ptrs
        d.tokens = tok
        d.steps = stp if stp is not None else ctypes.POINTER(ctypes.c_uint64)()
        d.quorum_mask = f["quorum_mask"] & (2**64 - 1)
        d.K = int(f["K"])
        d.n = int(f["n"])
    return descs, keep


NOALLOC_MAX_FRAGMENTS = 32


def merge_fragments_batched_noalloc(fragments, M: int, learner_dtype: int, outer_lr: float,
                                    outer_mu: float, *, flags: int = 0, records=None,
                                    stream=None) -> None:
    """``dd_merge_fragments_batched_noalloc``: the batched merge on the current
    device without a context and without any device allocation (at most
    ``NOALLOC_MAX_FRAGMENTS`` fragments; calls must not overlap on the GPU)."""
    descs, _keep = _pack_descs(fragments, M)
    rc = lib.dd_merge_fragments_batched_noalloc(
        descs, len(fragments), M, learner_dtype, ctypes.c_float(outer_lr),
        ctypes.c_float(outer_mu), ctypes.c_uint32(flags), _ptr(records), _stream_handle(stream))
    if rc != OK:
        raise DDMergeError(rc)


def _infer_dtype(learners) -> int:
    import torch
    if isinstance(learners, ctypes.Array):
        raise ValueError("learner_dtype must be given with a packed pointer array")
    for t in learners:
        if t is not None and not isinstance(t, int):
            return BF16 if t.dtype == torch.bfloat16 else F32
    return BF16


def launch_shape(learner_dtype: int, participants: int, pushed: int = 0, with_out_bf16: bool = False):
    """``dd_launch_shape``: (persistent CTAs per SM, ring slots per warp) of such a merge."""
    ctas, slots = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib.dd_launch_shape(int(learner_dtype), int(participants), int(pushed), int(bool(with_out_bf16)),
                             ctypes.byref(ctas), ctypes.byref(slots))
    if rc != OK:
        raise DDMergeError(rc)
    return ctas.value, slots.value


def select_quorum(arrival_s, K: int, grace_s: float):
    """``dd_select_quorum``: returns (mask, n_admitted)."""
    M = len(arrival_s)
    arr = (ctypes.c_double * M)(*[float(a) for a in arrival_s])
    mask, n_adm = ctypes.c_uint64(0), ctypes.c_int(0)
    rc = lib.dd_select_quorum(arr, M, int(K), float(grace_s), ctypes.byref(mask),
                              ctypes.byref(n_adm))
    if rc != OK:
        raise DDMergeError(rc)
    return int(mask.value), int(n_adm.value)


def grace_window(tau: float, xi_step: float, xi_quorum: float, xi_sync: float,
                 gamma: float) -> float:
    """``dd_grace_window``."""
    return float(lib.dd_grace_window(tau, xi_step, xi_quorum, xi_sync, gamma))


def plan_fragments(size_bits, layer, P: int, strategy: int):
    """``dd_plan_fragments``: returns (fragment index per tensor, total bits per fragment).
    ``layer`` holds the 0-based transformer layer of each tensor or -1 (may be None for
    FRAG_BALANCED)."""
    Q = len(size_bits)
    sizes = _u64_array(size_bits)
    lay = None if layer is None else (ctypes.c_int32 * Q)(*[int(x) for x in layer])
    out = (ctypes.c_int32 * max(Q, 1))()
    totals = (ctypes.c_uint64 * max(P, 1))()
    rc = lib.dd_plan_fragments(sizes, lay, Q, int(P), int(strategy), out, totals)
    if rc != OK:
        raise DDMergeError(rc)
    return [int(out[q]) for q in range(Q)], [int(totals[p]) for p in range(P)]


class GraceController:
    """``dd_grace_controller``: moving averages of step / quorum / sync durations and the
    grace window they allow."""

    def __init__(self, tau: float, gamma: float, beta: float):
        self._c = CGraceController()
        rc = lib.dd_grace_controller_init(ctypes.byref(self._c), tau, gamma, beta)
        if rc != OK:
            raise DDMergeError(rc)

    def observe(self, step_s: float, quorum_s: float, sync_s: float) -> None:
        rc = lib.dd_grace_controller_observe(ctypes.byref(self._c), step_s, quorum_s, sync_s)
        if rc != OK:
            raise DDMergeError(rc)

    def window(self) -> float:
        return float(lib.dd_grace_controller_window(ctypes.byref(self._c)))

    @property
    def averages(self):
        return self._c.xi_step, self._c.xi_quorum, self._c.xi_sync
