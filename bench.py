#!/usr/bin/env python
"""Benchmark of the fused per-fragment merge on B200.

One "step" is one pass of the whole hot path -- participation, weights, outer
gradients, weighted reduce, outer optimizer step, norm diagnostics -- over one
synthetic workload (default: one 500M-parameter fragment, 32 bf16 learner
copies of which 24 are in quorum, fp32 global + momentum).  Prints ONE JSON
line on rank 0.  At N = 1 the line also carries, under "configs", one row for
every other workload and merge kind (tiny, dense150m, dense1b3, moe4b, the
radial-directional and int4 merges of the headline workload, the syncer loop),
and, under roofline.same_run_ceilings, what this GPU gives probe kernels that
move data like the merge does but compute nothing.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --gpus 8               # starts 8 ranks itself, one per GPU
    python bench.py --gpus 8 --dry-launch  # prints the ranks' environments, runs nothing
    python bench.py --impl reference       # the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "merged_params_per_sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126e6
PROBE_SRC = os.path.join(ROOT, "bench_probes.cu")
PROBE_LIB = os.path.join(ROOT, "bench_probes.so")
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic_bytes_per_param.txt")


def host_cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.lower().startswith("model name"):
                    return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="scale500m")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink every fragment (profiling)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-ceilings", action="store_true",
                    help="skip the same-run bandwidth ceilings (probe kernels)")
    ap.add_argument("--configs", default="all",
                    help="N = 1: which other workloads get a row in the line's 'configs' array: "
                         "'all', 'none', or a comma-separated list of "
                         "tiny,dense150m,dense1b3,moe4b,rda,rda_dense150m,int4,push,broadcast,tape24")
    ap.add_argument("--config-steps", type=int, default=20, help="timed launches per 'configs' row")
    ap.add_argument("--cpu-sample", type=int, default=1 << 27,
                    help="elements of the workload the CPU oracle is timed on")
    ap.add_argument("--out-bf16", action="store_true", help="also write the bf16 broadcast copy")
    ap.add_argument("--unfused-push", action="store_true",
                    help="tape24: separate merge and broadcast launches instead of the fused push")
    ap.add_argument("--merge", choices=["avg", "rda", "int4"], default="avg",
                    help="weighted direct averaging (the headline path), radial-directional, or "
                         "direct averaging of int4-compressed outer gradients")
    ap.add_argument("--rda-three-pass", action="store_true",
                    help="--merge rda: force the three-launch form (norms, direction, apply) where the "
                         "two-launch form through the Gram matrix would be taken")
    ap.add_argument("--resident", choices=["all", "participants"], default="all",
                    help="allocate every learner copy, or only those that take part")
    ap.add_argument("--sharding", choices=["replica", "range"], default="replica",
                    help="N>1: every rank merges its own copy of the workload (weak scaling), or "
                         "each rank owns a contiguous element range of every fragment (strong)")
    ap.add_argument("--dry-launch", action="store_true",
                    help="print the environment and command of every rank --gpus N would start, then exit")
    return ap.parse_args(argv)


# ---- workload accounting (reporting only) ----------------------------------------------

def participants(w, p: int) -> int:
    """Learners of fragment p whose mask bit is set and whose token count is positive."""
    return sum(1 for m in range(w.M) if (w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0)


def bytes_per_param(merge: str, s: int, b_theta: int, out_bf16: bool = False, rda_three_pass: bool = False) -> float:
    """Algorithmic bytes per merged parameter: every participant's payload once, the global
    fragment and the momentum read once and written once.
      avg   s b + 16 (+ 2 with the bf16 copy)
      int4  s (1/2 + 4/128) + 16
      rda   the copies and Theta twice, Theta and v read and written, and the Gram products or the
            stored direction: see rda_bytes_per_param."""
    if merge == "int4":
        return s * (0.5 + 4.0 / 128.0) + 16 + (2 if out_bf16 else 0)
    if merge == "push":           # the merge, and Theta' written over every participant's copy
        return 2 * s * b_theta + 16
    if merge == "rda":
        return rda_bytes_per_param(s, b_theta, rda_three_pass) + (2 if out_bf16 else 0)
    return s * b_theta + 16 + (2 if out_bf16 else 0)


RDA_GRAM_MAX_PARTICIPANTS = 8


def rda_bytes_per_param(s: int, b_theta: int, three_pass: bool = False) -> float:
    """Up to 8 participants, two launches: the Gram matrix of the outer gradients (copies + Theta)
    and the ordinary merge (copies, Theta, v read; Theta, v written) = 2 s b + 20.  Otherwise three:
    norms (copies + Theta), direction (copies + Theta, write u), apply (Theta, v, u read; Theta, v
    written) = 2 (s b + 4) + 24."""
    if s <= RDA_GRAM_MAX_PARTICIPANTS and not three_pass:
        return 2 * s * b_theta + 20
    return 2 * (s * b_theta + 4) + 24


def rda_launches(w, three_pass: bool = False) -> int:
    gram = not three_pass and all(participants(w, p) <= RDA_GRAM_MAX_PARTICIPANTS for p in range(w.P))
    return 2 if gram else 3


def algorithmic_bytes(w, merge: str = "avg", out_bf16: bool = False, rda_three_pass: bool = False) -> int:
    b_theta = 2 if w.learner_dtype == "bf16" else 4
    three = merge == "rda" and rda_launches(w, rda_three_pass) == 3      # one form for the whole batch
    return int(sum(n * bytes_per_param(merge, participants(w, p), b_theta, out_bf16, three)
                   for p, n in enumerate(w.fragment_sizes)))


def write_share(w, merge: str = "avg", out_bf16: bool = False, rda_three_pass: bool = False) -> float:
    """Fraction of the algorithmic bytes that are writes."""
    total = algorithmic_bytes(w, merge, out_bf16, rda_three_pass)
    b_theta = 2 if w.learner_dtype == "bf16" else 4
    stored_direction = merge == "rda" and rda_launches(w, rda_three_pass) == 3
    writes = sum(n * (8 + (2 if out_bf16 else 0) + (4 if stored_direction else 0) +
                      (participants(w, p) * b_theta if merge == "push" else 0))
                 for p, n in enumerate(w.fragment_sizes))
    return writes / total if total else 0.0


def ncu_traffic_table():
    """(merge kind, workload) -> DRAM bytes per merged parameter measured by ncu
    (dram__bytes_read.sum + dram__bytes_write.sum); the file is written with the summaries
    under profiles/."""
    table = {}
    try:
        with open(TRAFFIC_FILE) as fh:
            for ln in fh:
                ln = ln.split("#", 1)[0].split()
                if len(ln) >= 3:
                    table[(ln[0], ln[1])] = float(ln[2])
    except OSError:
        pass
    return table


# ---- clocks ------------------------------------------------------------------------

_REASONS = {
    0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
    0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
    0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
}


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) in a thread."""

    def __init__(self, device_index: int, period_s: float = 0.01):
        self.period = period_s
        self.samples, self.reason_bits = [], 0
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.samples.append(mhz)
                self.reason_bits |= bits & ~0x1
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        reasons = [name for bit, name in _REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.samples)}


# ---- measured peaks and same-run ceilings ---------------------------------------------

def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def build_probes(force: bool = False) -> str:
    """Compiles bench_probes.cu (sm_100a) into bench_probes.so when missing or stale."""
    if not force and os.path.exists(PROBE_LIB) and os.path.getmtime(PROBE_LIB) >= os.path.getmtime(PROBE_SRC):
        return PROBE_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = PROBE_LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "--shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-o", tmp, PROBE_SRC]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
        raise RuntimeError("nvcc failed building bench_probes.so")
    os.replace(tmp, PROBE_LIB)
    return PROBE_LIB


class Probes:
    """The probe kernels of bench_probes.cu on one scratch buffer."""

    def __init__(self, device, scratch_bytes: int = 9 << 30):
        import torch
        self.lib = ctypes.CDLL(build_probes())
        self.lib.ddp_stream_probe.restype = ctypes.c_double
        self.lib.ddp_stream_probe.argtypes = [
            ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
            ctypes.POINTER(ctypes.c_double)]
        free = torch.cuda.mem_get_info(device)[0]
        self.bytes = int(min(scratch_bytes, max(1 << 30, free // 2)))
        self.buf = torch.empty(self.bytes, dtype=torch.uint8, device=device)
        self.buf.fill_(0x3c)
        self.stream = int(torch.cuda.current_stream().cuda_stream)

    def run(self, rd2=0, rd4=0, wr4=0, wr2=0, push_in_place=False, ctas_per_sm=2, ring_depth=3, reps=10):
        """GB/s of the shape (best of ``reps``), streams sized to fill the scratch buffer."""
        row_bytes = 2048 * (rd2 + (0 if push_in_place else wr2)) + 4096 * max(rd4, wr4)
        if push_in_place:
            row_bytes += 2048 * max(0, wr2 - rd2)
        rows = (self.bytes - (1 << 20)) // row_bytes
        ms = ctypes.c_double(0.0)
        gbs = self.lib.ddp_stream_probe(self.buf.data_ptr(), self.bytes, rd2, rd4, wr4, wr2,
                                        rows * 1024, int(push_in_place), ctas_per_sm, ring_depth, reps, self.stream,
                                        ctypes.byref(ms))
        if gbs < 0:
            raise RuntimeError(f"bandwidth probe failed (code {gbs})")
        return gbs

    def close(self):
        import torch
        del self.buf
        torch.cuda.empty_cache()


def measure_ceilings(device):
    """What this GPU gives, in this run, to kernels that move data the way the merge does but
    compute nothing (bench_probes.cu): a read-only stream set, a write-only one, and the
    headline mix; each over the whole scratch buffer (about 9 GB), best of 10."""
    pr = Probes(device)
    out = {
        "read_gbs": pr.run(rd2=24),
        "write_gbs": pr.run(wr4=2),
        "mix_gbs": pr.run(rd2=24, rd4=2, wr4=2),
        "how": "bench_probes.cu: 2 KB cp.async.bulk warp rings over 24 two-byte streams (read); "
               "st.global.cs.v8 into two four-byte streams (write); the merge's own pattern at "
               "24 participants, 87.5 % reads (mix); about 9 GB each, best of 10, CUDA events",
    }
    return out, pr


def merge_ring_depth(s: int, learner_dtype: str) -> int:
    """Ring slots the fused merge uses per warp at s participants, asked of the library
    (``dd_launch_shape``), so that a pattern probe moves data exactly as the kernel does."""
    from paper_2604_21428_b200 import ddmerge as dd
    return dd.launch_shape(dd.BF16 if learner_dtype == "bf16" else dd.F32, s)[1]


def push_launch_shape(s: int, k: int) -> tuple[int, int]:
    """(CTAs per SM, ring slots) of a merge of s bf16 copies fused with a push to k of them, asked
    of the library (``dd_launch_shape``)."""
    from paper_2604_21428_b200 import ddmerge as dd
    return dd.launch_shape(dd.BF16, s, k)


def blend_ceiling(read_gbs: float, write_gbs: float, wshare: float) -> float:
    """Bandwidth of a stream with the given share of writes if reads and writes each ran at
    their own ceiling and did not disturb one another (an upper bound, not a measurement)."""
    return 1.0 / ((1.0 - wshare) / read_gbs + wshare / write_gbs)


# ---- the reference arm: the CPU oracle ------------------------------------------------

def run_reference(args):
    """Times the oracle, as it stands, on the host cores: each step is one merge of a
    bounded sample (2^22 elements) of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2604_21428_b200 import synth

    w = synth.workload(args.workload)
    sample = min(1 << 22, w.fragment_sizes[0])
    p = 0
    part = [m for m in range(w.M) if (w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0]
    theta, v, learners = synth.fragment_cpu(sample, w.M, w.learner_dtype, w.seed, present=part)
    tokens = [int(x) for x in w.tokens[p]]
    oracle.build()
    for _ in range(min(args.warmup, 1)):
        oracle.merge_fragment(theta, v, learners, tokens, w.masks[p], w.K, synth.OUTER_LR,
                              synth.OUTER_MU)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.merge_fragment(theta, v, learners, tokens, w.masks[p], w.K, synth.OUTER_LR,
                              synth.OUTER_MU)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    sample_desc = (f"{sample} elements of fragment 0 of {w.name} per step, "
                   f"{len(part)} participating {w.learner_dtype} learners, single thread")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "sample_elements_per_step": sample, "M": w.M,
                   "participants": len(part), "learner_dtype": w.learner_dtype},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": sample_desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- starting the ranks -----------------------------------------------------------------

def _free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def launch_plan(n_ranks: int, argv, port: int | None = None):
    """Environment and command of every rank of a one-node job: one process per GPU."""
    port = port or _free_port()
    plan = []
    for r in range(n_ranks):
        env = {"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n_ranks),
               "LOCAL_WORLD_SIZE": str(n_ranks), "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)}
        plan.append({"rank": r, "env": env, "argv": [sys.executable, os.path.abspath(__file__)] + list(argv)})
    return plan


def spawn_ranks(args, argv) -> int:
    """``python bench.py --gpus N`` outside a launcher: starts the N ranks itself (what
    ``python -m torch.distributed.run --nproc-per-node N`` would do) and waits for them.  Rank 0
    prints the JSON line; the exit code is the first non-zero one."""
    import torch
    have = torch.cuda.device_count()
    if have < args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} asks for more GPUs than this node has ({have})\n")
        return 2
    plan = launch_plan(args.gpus, argv)
    procs = []
    for item in plan:
        procs.append(subprocess.Popen(item["argv"], env=dict(os.environ, **item["env"])))
    rc = 0
    try:
        pending = list(procs)
        while pending:
            for pr in list(pending):
                code = pr.poll()
                if code is None:
                    continue
                pending.remove(pr)
                if code != 0 and rc == 0:
                    rc = code
                    for other in pending:           # a rank failed: the others would wait for it forever
                        other.terminate()
            time.sleep(0.05)
    finally:
        for pr in procs:
            if pr.poll() is None:
                pr.kill()
    return rc


# ---- our arm ---------------------------------------------------------------------------

def build_workload(w, device, rank_seed, out_bf16, resident="all"):
    """Allocates and fills every fragment of workload ``w`` on ``device``."""
    import torch

    from paper_2604_21428_b200 import synth

    ldt = torch.bfloat16 if w.learner_dtype == "bf16" else torch.float32
    frags = []
    for p, n in enumerate(w.fragment_sizes):
        theta = torch.empty(n, dtype=torch.float32, device=device)
        mom = torch.empty(n, dtype=torch.float32, device=device)
        keep = [m for m in range(w.M)
                if resident == "all" or ((w.masks[p] >> m) & 1 and int(w.tokens[p, m]) > 0)]
        learners = [torch.empty(n, dtype=ldt, device=device) if m in keep else None
                    for m in range(w.M)]
        synth.fill_fragment_gpu(theta, mom, learners, seed=w.seed * 1000 + p + 100000 * rank_seed)
        out = torch.empty(n, dtype=torch.bfloat16, device=device) if out_bf16 else None
        frags.append(dict(global_=theta, momentum=mom, learners=learners, out_bf16=out,
                          tokens=[int(x) for x in w.tokens[p]], quorum_mask=w.masks[p], K=w.K, n=n))
    return frags


def resident_bytes(w, resident: str) -> int:
    b_theta = 2 if w.learner_dtype == "bf16" else 4
    copies = [w.M if resident == "all" else participants(w, p) for p in range(w.P)]
    return int(sum(n * (8 + c * b_theta) for n, c in zip(w.fragment_sizes, copies)))


class Merger:
    """One workload resident on the GPU and the library call that merges it."""

    def __init__(self, dd, ctx, w, device, *, merge="avg", out_bf16=False, resident="all", rank_seed=0,
                 frags=None, range_sharded_rda=False):
        import torch
        from paper_2604_21428_b200 import synth
        self.dd, self.ctx, self.w, self.merge, self.device = dd, ctx, w, merge, device
        self.frags = frags if frags is not None else build_workload(w, device, rank_seed, out_bf16, resident)
        self.ldtype = dd.BF16 if w.learner_dtype == "bf16" else dd.F32
        self.records = dd.new_records(w.P, device=device)
        self.flags = dd.DIAG_STATE
        self.eta, self.mu = synth.OUTER_LR, synth.OUTER_MU
        self.launches_per_step = 1
        self.push_mask = 0              # learners whose copy the merge overwrites with Theta' (fused push)
        self.int4_codes = self.int4_scales = None
        self.rda_scratch = None
        if merge == "int4":
            # the learners' side, outside every timed region: compress each participant's outer gradient
            assert w.P == 1, "the int4 merge takes a single-fragment workload"
            self.quantise()
        if merge == "rda":
            self.launches_per_step = 3 if range_sharded_rda else rda_launches(w)
            if range_sharded_rda:
                self.rda_scratch = torch.empty(sum((n + 7) // 8 * 8 for n in w.fragment_sizes),
                                               dtype=torch.float32, device=device)
        # the same buffers are merged every step: marshal their addresses and counts once
        self.packed_ptrs = dd.pack_pointers(self.frags[0]["learners"]) if w.P == 1 else None
        self.packed_tokens = dd.pack_u64(self.frags[0]["tokens"]) if w.P == 1 else None

    def quantise(self):
        import torch
        f, w = self.frags[0], self.w
        n0 = f["n"]
        self.int4_codes, self.int4_scales = [None] * w.M, [None] * w.M
        for m in range(w.M):
            if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0:
                self.int4_codes[m] = torch.empty((n0 + 1) // 2, dtype=torch.uint8, device=self.device)
                self.int4_scales[m] = torch.empty((n0 + 127) // 128, dtype=torch.float32, device=self.device)
                self.ctx.quantize_outer_gradient_int4(f["global_"], f["learners"][m], self.int4_codes[m],
                                                      self.int4_scales[m], n=n0, learner_dtype=self.ldtype)
        torch.cuda.synchronize()

    def step(self, stream=None):
        import torch
        from paper_2604_21428_b200 import dist as ddist
        ctx, w, f0 = self.ctx, self.w, self.frags[0]
        stream = stream if stream is not None else torch.cuda.current_stream()
        if self.merge == "int4":
            ctx.merge_fragment_int4(f0["global_"], f0["momentum"], self.int4_codes, self.int4_scales,
                                    f0["tokens"], f0["quorum_mask"], f0["K"], self.eta, self.mu, n=f0["n"],
                                    flags=self.flags, out_bf16=f0["out_bf16"], record=self.records,
                                    stream=stream)
        elif self.merge == "rda" and self.rda_scratch is not None:
            # range-sharded: the passes one by one, norms all-reduced over the ranks in between
            ddist.rda_merge_range_sharded(ctx, self.frags, w.M, self.ldtype, self.eta, self.mu,
                                          records=self.records, scratch=self.rda_scratch,
                                          flags=self.flags, stream=stream)
        elif self.merge == "rda":
            ctx.merge_fragments_batched_rda(self.frags, w.M, self.ldtype, self.eta, self.mu,
                                            flags=self.flags, records=self.records, stream=stream)
        elif w.P == 1 and self.push_mask:
            ctx.merge_fragment_push(f0["global_"], f0["momentum"], self.packed_ptrs, self.packed_tokens,
                                    f0["quorum_mask"], f0["K"], self.eta, self.mu, self.push_mask, n=f0["n"],
                                    learner_dtype=self.ldtype, flags=self.flags, record=self.records,
                                    stream=stream)
        elif w.P == 1:
            ctx.merge_fragment(f0["global_"], f0["momentum"], self.packed_ptrs, self.packed_tokens,
                               f0["quorum_mask"], f0["K"], self.eta, self.mu, n=f0["n"],
                               learner_dtype=self.ldtype, flags=self.flags, out_bf16=f0["out_bf16"],
                               record=self.records, stream=stream)
        else:
            ctx.merge_fragments_batched(self.frags, w.M, self.ldtype, self.eta, self.mu, flags=self.flags,
                                        records=self.records, stream=stream)

    # ---- parity evidence on the buffers that are about to be timed --------------------
    def first_merge_parity(self, max_fragments: int = 4):
        """Runs the FIRST merge (fresh state) and compares sampled 65,536-element windows of it
        with the oracle: inputs are copied out before the merge; nothing flows from the GPU into
        the oracle.  The int4 merge is checked end to end (the oracle quantises the window itself;
        windows start on block boundaries).  A radial-directional merge depends on whole-fragment
        norms, so a window cannot be given to the oracle: no windows, said so."""
        import numpy as np
        import torch

        import oracle
        w = self.w
        if self.merge == "rda":
            self.step()
            torch.cuda.synchronize()
            return {"windows": 0, "note": "radial-directional merge: whole-fragment norms, no window "
                                           "parity here; element-by-element parity is in tests/test_gpu_rda.py"}

        def host_learner(t):
            t = t.cpu()
            return t.view(torch.int16).numpy().view(np.uint16).copy() if t.dtype == torch.bfloat16 \
                else t.numpy().copy()

        picks = sorted(set([0, w.P - 1] + list(range(0, w.P, max(1, w.P // max_fragments)))))[:max_fragments + 1]
        saved = {}
        for p in picks:
            f = self.frags[p]
            n = f["n"]
            win = min(1 << 16, n)
            starts = sorted({0, max(0, (n - win) // 128 * 128), (n // 3) // 128 * 128, (2 * n // 3) // 128 * 128})
            starts = [s0 for s0 in starts if s0 + win <= n]
            part = [m for m in range(w.M) if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0]
            saved[p] = (win, starts, [(f["global_"][s0:s0 + win].cpu().numpy().copy(),
                                       f["momentum"][s0:s0 + win].cpu().numpy().copy(),
                                       [host_learner(f["learners"][m][s0:s0 + win]) if m in part else None
                                        for m in range(w.M)]) for s0 in starts])
        self.step()
        torch.cuda.synchronize()
        recs = self.dd.read_records(self.records)
        worst = {"t": 0.0, "v": 0.0}
        exact, nwin = True, 0
        pushed_ok, pushed_same = True, 1.0
        for p in picks:
            f, rec = self.frags[p], recs[p]
            win, starts, per = saved[p]
            for s0, (t0, v0, ls) in zip(starts, per):
                if self.merge == "int4":
                    q = [None if a is None else oracle.quantize_int4(t0, a) for a in ls]
                    ref = oracle.merge_fragment_int4(t0, v0, [None if x is None else x[0] for x in q],
                                                     [None if x is None else x[1] for x in q], f["tokens"],
                                                     f["quorum_mask"], f["K"], self.eta, self.mu)
                else:
                    ref = oracle.merge_fragment(t0, v0, ls, f["tokens"], f["quorum_mask"], f["K"],
                                                self.eta, self.mu)
                exact &= (rec.status, rec.n_part, rec.idx) == (ref.status, ref.n_part, ref.idx)
                exact &= rec.w_hat == [float(np.float32(x)) for x in ref.w_hat]
                if self.push_mask:
                    # every pushed copy now holds Theta' rounded to the learner dtype
                    want_bits = oracle.bf16_rne(t0)
                    for m in range(w.M):
                        if (self.push_mask >> m) & 1:
                            pushed_ok &= bool(np.array_equal(host_learner(f["learners"][m][s0:s0 + win]),
                                                             oracle.bf16_rne(f["global_"][s0:s0 + win].cpu().numpy())))
                            same = np.mean(host_learner(f["learners"][m][s0:s0 + win]) == want_bits)
                            pushed_same = min(pushed_same, float(same))
                for got, want, which in ((f["global_"], t0, "t"), (f["momentum"], v0, "v")):
                    g = got[s0:s0 + win].cpu().numpy().astype(np.float64)
                    o = want.astype(np.float64)
                    rms = float(np.sqrt(np.mean(o * o))) or 1.0
                    worst[which] = max(worst[which], float(np.max(np.abs(g - o) / np.maximum(np.abs(o), rms))))
                nwin += 1
        out = {"windows": nwin, "window_elems": saved[picks[0]][0], "fragments_sampled": len(picks),
               "max_err_theta": worst["t"], "max_err_momentum": worst["v"], "tolerance": 1e-5,
               "participation_and_weights_bit_exact": bool(exact),
               "metric": "first merge: max |gpu - oracle| / max(|oracle|, rms(oracle))"}
        if self.push_mask:
            out["pushed_copies_equal_rounded_theta"] = bool(pushed_ok)
            out["pushed_bits_equal_to_oracle_fraction_min"] = pushed_same
        return out

    def timed(self, steps: int, warmup: int, world: int = 1):
        """``warmup`` untimed steps, then ``steps`` timed ones bracketed by a barrier and a
        synchronize on both sides; one CUDA event after every step gives the per-launch times."""
        import torch
        import torch.distributed as dist
        stream = torch.cuda.current_stream()
        for _ in range(max(warmup, 3)):
            self.step()
        torch.cuda.synchronize()
        recs = self.dd.read_records(self.records)
        assert all(r.status == 0 for r in recs), [r.status for r in recs]
        sampler = ClockSampler(self.device.index or 0)
        events = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.start()
        events[0].record(stream)
        for k in range(steps):
            self.step()
            events[k + 1].record(stream)
        torch.cuda.synchronize()
        sampler.stop()
        if world > 1:
            dist.barrier()
        total_ms = events[0].elapsed_time(events[-1])
        per_launch_ms = [events[k].elapsed_time(events[k + 1]) for k in range(steps)]
        return total_ms, per_launch_ms, sampler.summary()

    def timed_cold(self, steps: int):
        """A workload that fits in L2 is also timed cold: a 512 MB buffer is rewritten between
        launches and only the merge is bracketed by events."""
        import torch
        stream = torch.cuda.current_stream()
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=self.device)
        cold = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for k in range(steps):
            flush.fill_(k & 0xff)
            e0.record(stream)
            self.step()
            e1.record(stream)
            e1.synchronize()
            cold.append(e0.elapsed_time(e1))
        del flush
        return {"median": statistics.median(cold), "min": min(cold), "max": max(cold)}

    def timed_graph(self, reps: int = 50):
        """A single small fragment is launch-bound from Python (the host needs longer to issue a
        merge than the GPU to run it): the same calls captured once into a CUDA graph and
        replayed give the device-bound time per merge.  The single-fragment call is capture-safe
        (one kernel launch, no allocation or synchronisation once the workspace exists)."""
        import torch
        side = torch.cuda.Stream(device=self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for _ in range(reps):
                    self.step(side)
        torch.cuda.synchronize()
        times = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(8):
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1) / reps)
        del graph
        return {"median": statistics.median(times[3:]), "min": min(times[3:]), "merges_per_graph": reps}

    def timed_prepared(self, reps: int = 200):
        """The same single-fragment merges issued through ``prepare_merge_fragment`` (arguments
        marshalled once): what a host loop that calls the library directly pays per merge."""
        import torch
        f0 = self.frags[0]
        stream = torch.cuda.current_stream()
        call = self.ctx.prepare_merge_fragment(
            f0["global_"], f0["momentum"], self.packed_ptrs, self.packed_tokens, f0["K"], self.eta, self.mu,
            n=f0["n"], learner_dtype=self.ldtype, flags=self.flags, out_bf16=f0["out_bf16"],
            record=self.records, stream=stream)
        mask = f0["quorum_mask"]
        for _ in range(20):
            call(mask)
        times = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(5):
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(reps):
                call(mask)
            e1.record(stream)
            e1.synchronize()
            times.append(e0.elapsed_time(e1) / reps)
        return {"median": statistics.median(times), "min": min(times), "merges_per_sample": reps}

    def free(self):
        import torch
        self.frags = self.int4_codes = self.int4_scales = self.rda_scratch = self.records = None
        self.packed_ptrs = None
        torch.cuda.empty_cache()


def roofline_of(w, merge, out_bf16, per_launch_ms, ceilings, traffic_table, workload_name, rda_three_pass=False):
    """The roofline object of one timed workload (HBM-bound; no tensor cores on this path)."""
    alg = algorithmic_bytes(w, merge, out_bf16, rda_three_pass)
    avg = sum(per_launch_ms) / len(per_launch_ms)
    achieved = alg / (avg * 1e-3) / 1e9
    peak, peak_kind = hbm_peak()
    tpp = None if out_bf16 else traffic_table.get((merge, workload_name))
    r = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "peak_source": f"of {peak_kind}",
        "traffic": None if tpp is None else tpp * w.total_params,
        "algorithmic_bytes_per_launch": alg, "bytes_per_param": alg / w.total_params,
        "write_share": write_share(w, merge, out_bf16, rda_three_pass),
        "kernel_ms": {"avg": avg, "median": statistics.median(per_launch_ms), "min": min(per_launch_ms),
                      "max": max(per_launch_ms)},
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
    }
    if ceilings:
        blend = blend_ceiling(ceilings["read_gbs"], ceilings["write_gbs"], r["write_share"])
        r["frac_of_read_ceiling"] = achieved / ceilings["read_gbs"]
        r["blend_ceiling_gbs"] = blend
        r["frac_of_blend_ceiling"] = achieved / blend
    return r


def config_row(dd, ctx, device, name, merge, args, ceilings, probes, traffic_table, merger=None,
               resident="all"):
    """One row of the line's 'configs' array: a workload merged ``--config-steps`` times."""
    import torch

    from paper_2604_21428_b200 import synth
    w = merger.w if merger is not None else synth.workload(name)
    own = merger is None
    note = None
    if own:
        free = torch.cuda.mem_get_info(device)[0]
        if resident_bytes(w, resident) + (3 << 30) > free:
            resident = "participants"
        if resident_bytes(w, resident) + (3 << 30) > free:
            return {"workload": name, "merge": merge, "skipped":
                    f"needs {resident_bytes(w, resident) >> 30} GiB resident, {free >> 30} GiB free"}
        if resident == "participants":
            note = "only the participating learner copies are resident (the others are never read)"
        merger = Merger(dd, ctx, w, device, merge=merge, resident=resident)
    else:
        # another merge kind on buffers that are already resident: back to the seeded state first, so
        # that the parity windows below are again those of a FIRST merge
        merger.merge = "avg" if merge == "push" else merge
        merger.push_mask = merger.frags[0]["quorum_mask"] if merge == "push" else 0
        merger.launches_per_step = rda_launches(w) if merge == "rda" else 1
        for p, f in enumerate(merger.frags):
            synth.fill_fragment_gpu(f["global_"], f["momentum"], f["learners"], seed=w.seed * 1000 + p)
        if merge == "int4":
            merger.quantise()
    row = {"workload": name, "merge": merge, "fragments": w.P, "params": w.total_params, "M": w.M,
           "participants": [participants(w, p) for p in range(w.P)], "learner_dtype": w.learner_dtype}
    if note:
        row["note"] = note
    try:
        if not args.no_cpu_baseline:
            row["parity"] = merger.first_merge_parity()
        _, per_launch, clocks = merger.timed(args.config_steps, 3)
        r = roofline_of(w, merge, False, per_launch, ceilings, traffic_table, name)
        if merge == "push":
            row["note"] = "the merge also overwrites every participant's copy with Theta' (fused push, in place)" 
        row.update({
            "ms": r["kernel_ms"], "params_per_s": w.total_params / (r["kernel_ms"]["avg"] * 1e-3),
            "bytes_per_param": r["bytes_per_param"], "write_share": r["write_share"],
            "achieved_gbs": r["achieved"], "frac": r["frac"], "frac_of_nominal_8TBs": r["frac_of_nominal_8TBs"],
            "launches_per_merge": merger.launches_per_step, "steps": args.config_steps,
            "sm_mhz": clocks["sm_mhz"], "clock_reasons": clocks["reasons"],
            "traffic_bytes_per_param_ncu": traffic_table.get((merge, name)),
        })
        for k in ("frac_of_read_ceiling", "blend_ceiling_gbs", "frac_of_blend_ceiling"):
            if k in r:
                row[k] = r[k]
        alg = r["algorithmic_bytes_per_launch"]
        if alg < 4 * L2_BYTES:
            row["l2"] = "fits L2: 'ms' is warm (back to back); cold = 512 MB flush between launches"
            row["ms_l2_flushed"] = merger.timed_cold(min(args.config_steps, 20))
            row["achieved_gbs_l2_flushed"] = alg / (row["ms_l2_flushed"]["median"] * 1e-3) / 1e9
            if w.P == 1 and merge == "avg":
                row["ms_cuda_graph_replay"] = merger.timed_graph()
                row["ms_prepared_call"] = merger.timed_prepared()
        else:
            row["l2"] = "inputs larger than L2 (no flush)"
        if not args.no_e2e and merge in ("avg", "int4") and not (merge == "avg" and not own):
            # end to end from pinned host memory; the large workloads stream a bounded slice
            row["e2e"] = e2e_leg(dd, ctx, merger, args, 1, pinned_cap_bytes=12 << 30, steps=2)
        if probes is not None and merge == "push" and w.learner_dtype == "bf16":
            s_all = row["participants"][0]
            ctas, depth = push_launch_shape(s_all, s_all)
            row["pattern_probe_gbs"] = probes.run(rd2=s_all, rd4=2, wr4=2, wr2=s_all, push_in_place=True,
                                                  ctas_per_sm=ctas, ring_depth=depth, reps=5)
            row["frac_of_pattern_probe"] = row["achieved_gbs"] / row["pattern_probe_gbs"]
        if probes is not None and merge == "rda" and w.learner_dtype == "bf16":
            # one probe per launch of the merge (the same streams, nothing computed), added up
            s_mean = max(1, round(sum(row["participants"]) / w.P))
            depth = merge_ring_depth(s_mean, "bf16")
            if merger.launches_per_step == 2:
                legs = [("gram", 2 * s_mean + 4, dict(rd2=s_mean, rd4=1)),
                        ("merge", 2 * s_mean + 16, dict(rd2=s_mean, rd4=2, wr4=2, ring_depth=depth))]
            else:
                legs = [("norms", 2 * s_mean + 4, dict(rd2=s_mean, rd4=1, ring_depth=depth)),
                        ("direction", 2 * s_mean + 8, dict(rd2=s_mean, rd4=1, wr4=1, ring_depth=depth)),
                        # u, Theta, v read (u stands in as two two-byte streams), Theta', v' written
                        # (one CTA per SM with the full ring: the launcher's shape for this pass)
                        ("apply", 20, dict(rd2=2, rd4=2, wr4=2, ctas_per_sm=1, ring_depth=3))]
            t_total, b_total, per_leg = 0.0, 0.0, {}
            for leg, bpp, shape in legs:
                gbs = probes.run(reps=5, **shape)
                per_leg[leg] = gbs
                t_total += bpp / gbs
                b_total += bpp
            row["pattern_probe_gbs"] = b_total / t_total
            row["pattern_probe_per_launch_gbs"] = per_leg
            row["frac_of_pattern_probe"] = row["achieved_gbs"] / row["pattern_probe_gbs"]
        if probes is not None and merge == "avg":
            # the same access pattern with the arithmetic left out, at this workload's mean participant count
            s_mean = max(1, round(sum(row["participants"]) / w.P))
            if w.learner_dtype == "bf16":
                row["pattern_probe_gbs"] = probes.run(rd2=s_mean, rd4=2, wr4=2,
                                                      ring_depth=merge_ring_depth(s_mean, "bf16"), reps=5)
                row["frac_of_pattern_probe"] = row["achieved_gbs"] / row["pattern_probe_gbs"]
    finally:
        if own:
            merger.free()
    return row


def broadcast_row(dd, ctx, merger, args, ceilings, probes):
    """The learner side alone: Theta' read once and written (alpha = 0) over every participant's copy."""
    import numpy as np
    import torch

    import oracle
    w, f = merger.w, merger.frags[0]
    n = f["n"]
    mask = f["quorum_mask"]
    k = participants(w, 0)
    stream = torch.cuda.current_stream()

    def step():
        ctx.broadcast_fragment(f["global_"], merger.packed_ptrs, mask, 0.0, n=n, learner_dtype=merger.ldtype,
                               stream=stream)
    for _ in range(3):
        step()
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.config_steps + 1)]
    torch.cuda.synchronize()
    events[0].record(stream)
    for i in range(args.config_steps):
        step()
        events[i + 1].record(stream)
    torch.cuda.synchronize()
    ms = [events[i].elapsed_time(events[i + 1]) for i in range(args.config_steps)]
    esz = 2 if w.learner_dtype == "bf16" else 4
    alg = n * (4 + k * esz)
    avg = sum(ms) / len(ms)
    peak, _ = hbm_peak()
    row = {"workload": w.name, "merge": "broadcast", "fragments": 1, "params": n, "M": w.M, "copies_written": k,
           "learner_dtype": w.learner_dtype,
           "ms": {"avg": avg, "median": statistics.median(ms), "min": min(ms), "max": max(ms)},
           "params_per_s": n / (avg * 1e-3), "bytes_per_param": alg / n, "write_share": k * esz / (4 + k * esz),
           "achieved_gbs": alg / (avg * 1e-3) / 1e9, "frac": alg / (avg * 1e-3) / 1e9 / peak,
           "frac_of_nominal_8TBs": alg / (avg * 1e-3) / 1e9 / NOMINAL_HBM_GBS, "launches_per_merge": 1,
           "steps": args.config_steps, "l2": "inputs larger than L2 (no flush)",
           "note": "dd_broadcast_fragment, alpha = 0: the learner side of a syncer update on its own"}
    row["traffic_bytes_per_param_ncu"] = ncu_traffic_table().get(("broadcast", w.name))
    if ceilings:
        blend = blend_ceiling(ceilings["read_gbs"], ceilings["write_gbs"], row["write_share"])
        row["blend_ceiling_gbs"] = blend
        row["frac_of_blend_ceiling"] = row["achieved_gbs"] / blend
        row["frac_of_write_ceiling"] = row["achieved_gbs"] / ceilings["write_gbs"]
    if probes is not None and w.learner_dtype == "bf16":
        row["pattern_probe_gbs"] = probes.run(rd4=1, wr2=k, reps=5)
        row["frac_of_pattern_probe"] = row["achieved_gbs"] / row["pattern_probe_gbs"]
    if not args.no_cpu_baseline:
        # a window of every written copy against the oracle's rounding of the same Theta'
        win = min(1 << 16, n)
        want = oracle.bf16_rne(f["global_"][:win].cpu().numpy()) if esz == 2 else f["global_"][:win].cpu().numpy()
        ok = True
        for m in range(w.M):
            if (mask >> m) & 1:
                got = f["learners"][m][:win].cpu()
                got = got.view(torch.int16).numpy().view(np.uint16) if esz == 2 else got.numpy()
                ok &= bool(np.array_equal(got, want))
        row["parity"] = {"windows": k, "window_elems": win, "copies_bit_equal_to_oracle_rounding": ok}
    return row


def run_replay(args, ceilings=None):
    """Second workload: the syncer loop itself.  A 1.34B-parameter dense decoder (24 layers,
    d 2048, d_ff 8192) is cut into P = H = 24 balanced fragments by the library's planner;
    8 bf16 learners, K = 1, grace window of a quarter step; every syncer step merges the
    fragment that is due (one launch) and broadcasts it to the learners that are up, driven
    by a seeded synthetic event tape.  One bench step = one syncer step."""
    import torch

    from paper_2604_21428_b200 import build as lib_build
    lib_build.build()            # no-op when libddmerge.so is newer than its sources
    from paper_2604_21428_b200 import ddmerge as dd
    from paper_2604_21428_b200 import synth
    from paper_2604_21428_b200.replay import Syncer, TapeEntry

    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    M, P, H, K = 8, 24, 24, 1
    d_model = 2048
    if args.scale != 1.0:            # a smaller model of the same shape (profiling captures)
        d_model = max(64, int(2048 * args.scale ** 0.5) // 64 * 64)
    tensors = synth.dense_tensor_list(24, d_model, 4 * d_model, 32000)
    frag_of, bits = dd.plan_fragments([16 * n for n, _ in tensors], None, P, dd.FRAG_BALANCED)
    sizes = [b // 16 for b in bits]
    offsets = list(range(P))
    total_steps = args.warmup + args.steps
    tape = synth.synthetic_tape(M, P, H, offsets, total_steps, seed=11)
    theta = [torch.empty(n, dtype=torch.float32, device=device) for n in sizes]
    mom = [torch.empty(n, dtype=torch.float32, device=device) for n in sizes]
    learners = [[None] * P for _ in range(M)]
    for p, n in enumerate(sizes):
        copies = [torch.empty(n, dtype=torch.bfloat16, device=device) for _ in range(M)]
        synth.fill_fragment_gpu(theta[p], mom[p], copies, seed=7000 + p)
        for m in range(M):
            learners[m][p] = copies[m]
    ctx = dd.Context(0)
    syncer = Syncer(ctx, theta, mom, H=H, offsets=offsets, K=K, outer_lr=synth.OUTER_LR,
                    outer_mu=synth.OUTER_MU, learner_dtype=dd.BF16, flags=dd.DIAG_STATE,
                    fused_push=not args.unfused_push)
    stream = torch.cuda.current_stream()
    entries = [TapeEntry(arrival_s=e["arrival_s"], tokens=e["tokens"], steps=e["steps"]) for e in tape]
    for t in range(args.warmup):
        syncer.step(t, entries[t], learners, grace_s=0.25, stream=stream, read_back=False)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    merged_params = merged_bytes = written_bytes = launches = 0
    sampler.start()
    ev0.record(stream)
    for t in range(args.warmup, total_steps):
        res = syncer.step(t, entries[t], learners, grace_s=0.25, stream=stream, read_back=False)
        alive = sum(1 for a in entries[t].arrival_s if a != float("inf"))
        for p in res.due:
            s_p = sum(1 for m in range(M) if (res.mask >> m) & 1 and entries[t].tokens[p][m] > 0)
            if s_p >= max(K, 1):
                merged_params += sizes[p]
                # merge (read s copies, Theta, v; write Theta', v') + push (write the alive copies);
                # the unfused form reads Theta' once more in its broadcast launch
                merged_bytes += sizes[p] * (2 * s_p + 16) + sizes[p] * (2 * alive)
                written_bytes += sizes[p] * (8 + 2 * alive)
                if not syncer.fused_push:
                    merged_bytes += sizes[p] * 4
                    launches += 1
            launches += 1
    ev1.record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    ms = ev0.elapsed_time(ev1)
    peak, peak_kind = hbm_peak()
    achieved = merged_bytes / (ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": f"of {peak_kind}", "traffic": None,
                "algorithmic_bytes": merged_bytes, "write_share": written_bytes / max(merged_bytes, 1),
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                "note": ("merge and push fused in one launch per syncer step" if syncer.fused_push else
                         "merge + broadcast launches of the syncer loop") + ", host work included"}
    if ceilings:
        blend = blend_ceiling(ceilings["read_gbs"], ceilings["write_gbs"], roofline["write_share"])
        roofline["blend_ceiling_gbs"] = blend
        roofline["frac_of_blend_ceiling"] = achieved / blend
    line = {
        "metric": METRIC, "value": merged_params / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "tape24" if args.scale == 1.0 else f"tape24@{args.scale:g}",
                   "model_params": sum(sizes), "d_model": d_model, "fragments": P, "H": H, "M": M,
                   "K": K, "grace_s": 0.25, "fragment_elems_min_max": [min(sizes), max(sizes)],
                   "planner": "balanced", "learner_dtype": "bf16",
                   "l2": "inputs larger than L2 (no flush)"},
        "clocks": sampler.summary(), "gpu_launches": launches,
        "roofline": roofline,
        "e2e": None, "cpu_baseline": None,
    }
    ctx.close()
    del syncer, theta, mom, learners
    torch.cuda.empty_cache()
    return line


def e2e_leg(dd, ctx, merger, args, world, pinned_cap_bytes=None, steps=None):
    """End to end through the public host-buffer calls: pinned host buffers in, results in host
    memory, host<->device copies inside the timed region.  One fragment of learner copies goes
    through dd_merge_fragment_host, several through dd_merge_fragments_batched_host, int4 payloads
    through dd_merge_fragment_int4_host."""
    import torch
    import torch.distributed as dist

    from paper_2604_21428_b200 import dist as ddist
    w = merger.w
    steps = steps or args.e2e_steps
    int4 = merger.merge == "int4"
    esz = 2 if w.learner_dtype == "bf16" else 4
    parts = [[m for m in range(w.M) if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0] for f in merger.frags]

    def in_bytes(p, n):       # host-to-device bytes of n elements of fragment p
        if int4:
            return len(parts[p]) * ((n + 1) // 2 + (n + 127) // 128 * 4) + 8 * n
        return n * (len(parts[p]) * esz + 8)

    # Page-locked host memory is bounded: every rank of the node pins its own buffers, so with
    # several ranks (or little free host memory, or a cap given by the caller) the end-to-end leg
    # streams a leading slice of every fragment instead of all of it.
    try:
        avail = next(int(l.split()[1]) * 1024 for l in open("/proc/meminfo") if l.startswith("MemAvailable"))
    except Exception:
        avail = 64 << 30
    local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
    budget = int(0.4 * avail / max(local_world, 1))
    if pinned_cap_bytes:
        budget = min(budget, pinned_cap_bytes)
    full = sum(in_bytes(p, f["n"]) for p, f in enumerate(merger.frags))
    share = min(1.0, budget / max(full, 1))
    align = 128 if int4 else 8
    sizes = [max(align, int(f["n"] * share) // align * align) if share < 1.0 else f["n"] for f in merger.frags]
    host_frags, h2d, d2h = [], 0, 0
    for p, (f, n) in enumerate(zip(merger.frags, sizes)):
        h_theta = torch.empty(n, dtype=torch.float32, pin_memory=True)
        h_mom = torch.empty(n, dtype=torch.float32, pin_memory=True)
        h_theta.copy_(f["global_"][:n])
        h_mom.copy_(f["momentum"][:n])
        hf = dict(global_=h_theta, momentum=h_mom, tokens=f["tokens"], quorum_mask=f["quorum_mask"], K=f["K"], n=n)
        if int4:
            hf["codes"], hf["scales"] = [None] * w.M, [None] * w.M
            for m in parts[p]:
                hf["codes"][m] = torch.empty((n + 1) // 2, dtype=torch.uint8, pin_memory=True)
                hf["codes"][m].copy_(merger.int4_codes[m][:(n + 1) // 2])
                hf["scales"][m] = torch.empty((n + 127) // 128, dtype=torch.float32, pin_memory=True)
                hf["scales"][m].copy_(merger.int4_scales[m][:(n + 127) // 128])
        else:
            hf["learners"] = [None] * w.M
            for m in parts[p]:
                hf["learners"][m] = torch.empty(n, dtype=f["learners"][m].dtype, pin_memory=True)
                hf["learners"][m].copy_(f["learners"][m][:n])
        host_frags.append(hf)
        h2d += in_bytes(p, n)
        d2h += n * 8 + dd.RECORD_BYTES

    def one_step():
        if int4:
            hf = host_frags[0]
            return [ctx.merge_fragment_int4_host(hf["global_"], hf["momentum"], hf["codes"], hf["scales"],
                                                 hf["tokens"], hf["quorum_mask"], hf["K"], merger.eta, merger.mu,
                                                 n=hf["n"], flags=merger.flags)]
        if w.P == 1:
            hf = host_frags[0]
            return [ctx.merge_fragment_host(hf["global_"], hf["momentum"], hf["learners"], hf["tokens"],
                                            hf["quorum_mask"], hf["K"], merger.eta, merger.mu, n=hf["n"],
                                            learner_dtype=merger.ldtype, flags=merger.flags)]
        return ctx.merge_fragments_batched_host(host_frags, w.M, merger.ldtype, merger.eta, merger.mu,
                                                flags=merger.flags)

    steps = max(1, steps)
    # what the bus gives to a plain copy from page-locked memory in this run (256 MB, best of 3):
    # the end-to-end rate can at most be this divided by the bytes that cross per element
    probe_h = torch.empty(256 << 20, dtype=torch.uint8, pin_memory=True)
    probe_d = torch.empty(256 << 20, dtype=torch.uint8, device=merger.device)
    h2d_probe = 0.0
    for _ in range(4):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        probe_d.copy_(probe_h, non_blocking=True)
        torch.cuda.synchronize()
        h2d_probe = max(h2d_probe, probe_h.numel() / (time.perf_counter() - t0) / 1e9)
    del probe_h, probe_d

    one_step()                                           # warm-up: staging buffers, streams
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        recs = one_step()
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert all(r.status == 0 for r in recs)
    dt_max = ddist.max_over_ranks(dt, device=merger.device)
    n_total = sum(sizes)
    call = ("dd_merge_fragment_int4_host" if int4 else
            "dd_merge_fragment_host" if w.P == 1 else "dd_merge_fragments_batched_host")
    # every rank streams its own copy (or its own range) of the elements per step
    out = {"value": n_total * world * steps / dt_max, "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "steps": steps, "elements_per_rank_step": n_total,
           "h2d_gbs": h2d * steps / dt_max / 1e9,
           "h2d_copy_probe_gbs": h2d_probe,
           "frac_of_h2d_copy_probe": h2d * steps / dt_max / 1e9 / h2d_probe,
           "path": f"{call}: pinned host buffers, chunked H2D -> kernel -> D2H pipeline, blocking"}
    if share < 1.0:
        out["note"] = f"leading {share:.3f} of every fragment (page-locked host memory is bounded)"
    del host_frags
    return out


def cpu_baseline_leg(merger, args):
    """The oracle as it stands on the host cores, on a bounded sample of the same workload."""
    import numpy as np
    import torch

    import oracle
    w, f = merger.w, merger.frags[0]
    ns = min(args.cpu_sample, f["n"])
    part = [m for m in range(w.M) if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0]
    theta = f["global_"][:ns].cpu().numpy()
    mom = f["momentum"][:ns].cpu().numpy()
    learners = [None] * w.M
    for m in part:
        t_m = f["learners"][m][:ns].cpu()
        learners[m] = (t_m.view(torch.int16).numpy().view(np.uint16)
                       if w.learner_dtype == "bf16" else t_m.numpy())
    oracle.build()
    t0 = time.perf_counter()
    oracle.merge_fragment(theta, mom, learners, f["tokens"], f["quorum_mask"], f["K"], merger.eta, merger.mu)
    dt = time.perf_counter() - t0
    out = {"value": ns / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"first {ns} elements of fragment 0 of {w.name}, {len(part)} participating "
                     f"{w.learner_dtype} learners, one merge, {dt:.1f} s, single thread of "
                     f"{os.cpu_count()} host cores",
           "host_cpu": host_cpu_model(), "host_cores": os.cpu_count(),
           "affinity_cores": len(os.sched_getaffinity(0))}
    # Beside it, because the paper's own syncer is a CPU program: the same element loop
    # spread over all host cores (OpenMP; not the checked oracle, a timing baseline only).
    try:
        cores = len(os.sched_getaffinity(0))
        t0 = time.perf_counter()
        oracle.merge_fragment_all_cores(theta, mom, learners, f["tokens"], f["quorum_mask"], f["K"],
                                        merger.eta, merger.mu)
        dt_all = time.perf_counter() - t0
        out["all_cores"] = {"value": ns / dt_all, "unit": UNIT, "cores": cores,
                            "kind": "oracle element loop under OpenMP", "seconds": dt_all}
    except Exception as exc:      # no OpenMP runtime on the box: the oracle figure stands alone
        out["all_cores"] = {"unavailable": str(exc)[:120]}
    return out


def wanted_configs(args, headline, headline_merge):
    names = ["tiny", "dense150m", "dense1b3", "moe4b", "rda", "rda_dense150m", "int4", "push", "broadcast", "tape24"]
    if args.configs == "none":
        return []
    if args.configs != "all":
        asked = [x.strip() for x in args.configs.split(",") if x.strip()]
        bad = [x for x in asked if x not in names]
        if bad:
            raise SystemExit(f"--configs: unknown {bad}; choose from {names}")
        names = [x for x in names if x in asked]
    return [x for x in names if not (x == headline and headline_merge == "avg")]


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2604_21428_b200 import build as lib_build
    lib_build.build()            # no-op when libddmerge.so is newer than its sources
    from paper_2604_21428_b200 import ddmerge as dd
    from paper_2604_21428_b200 import dist as ddist
    from paper_2604_21428_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
        world = dist.get_world_size()            # the world that really initialised

    traffic_table = ncu_traffic_table()
    ceilings = probes = None
    if not args.no_ceilings:
        if rank == 0:
            build_probes()
        if world > 1:
            dist.barrier()
        ceilings, probes = measure_ceilings(device)

    if args.workload == "tape24":
        line = run_replay(args, ceilings)
        if ceilings:
            line["roofline"]["same_run_ceilings"] = ceilings
        if probes is not None:
            probes.close()
        print(json.dumps(line), flush=True)
        return

    w = synth.workload(args.workload)
    if args.scale != 1.0:
        w = synth.scaled(w, args.scale, align=8)
    job_params = w.total_params * (world if args.sharding == "replica" else 1)
    if args.sharding == "range" and world > 1:
        # int4 scales cover blocks of 128 elements: shard on block boundaries so that the sharded
        # job quantises exactly the blocks the unsharded one would
        align = 128 if args.merge == "int4" else 8
        w.fragment_sizes = [hi - lo for lo, hi in
                            (ddist.shard_range(n, rank, world, align) for n in w.fragment_sizes)]
    if probes is not None and resident_bytes(w, args.resident) + (4 << 30) > torch.cuda.mem_get_info(device)[0]:
        probes.close()                           # the workload needs the room of the probes' scratch buffer
        probes = None
    ctx = dd.Context(local_rank)
    merger = Merger(dd, ctx, w, device, merge=args.merge, out_bf16=args.out_bf16, resident=args.resident,
                    rank_seed=rank, range_sharded_rda=args.merge == "rda" and args.sharding == "range" and world > 1)
    three_pass = args.merge == "rda" and (args.rda_three_pass or (args.sharding == "range" and world > 1))
    if args.rda_three_pass:
        merger.flags |= dd.RDA_THREE_PASS
        merger.launches_per_step = 3
    grid, block, tile = ctx.launch_geometry(merger.ldtype)

    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        parity = merger.first_merge_parity()

    total_ms, per_launch_ms, clocks = merger.timed(args.steps, args.warmup, world)
    max_ms = ddist.max_over_ranks(total_ms, device=device)
    value = ddist.whole_job_rate(job_params, args.steps, 1, max_ms)
    roofline = roofline_of(w, args.merge, args.out_bf16, per_launch_ms, ceilings, traffic_table, args.workload,
                           three_pass)
    roofline["kernel_ms"]["slowest_steps"] = sorted(range(len(per_launch_ms)), key=lambda k: -per_launch_ms[k])[:3]
    alg_bytes = roofline["algorithmic_bytes_per_launch"]
    fits_l2 = alg_bytes < 4 * L2_BYTES
    if fits_l2:
        roofline["kernel_ms_l2_flushed"] = merger.timed_cold(min(args.steps, 20))
        roofline["achieved_l2_flushed"] = alg_bytes / (roofline["kernel_ms_l2_flushed"]["median"] * 1e-3) / 1e9
        if w.P == 1 and args.merge == "avg":
            roofline["ms_per_merge_cuda_graph_replay"] = merger.timed_graph()
    if ceilings:
        roofline["same_run_ceilings"] = ceilings
        roofline["frac_of_mix_ceiling"] = roofline["achieved"] / ceilings["mix_gbs"]

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": max_ms / args.steps, "higher_is_better": True,
        "scaling": "weak" if args.sharding == "replica" else "strong", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": w.name, "fragments": w.P, "params_per_step": w.total_params, "M": w.M,
            "participants": [participants(w, p) for p in range(w.P)],
            "learner_dtype": w.learner_dtype, "state_dtype": "f32", "outer_lr": merger.eta,
            "outer_mu": merger.mu, "flags": "nesterov+diag_state", "out_bf16": bool(args.out_bf16),
            "merge": args.merge,
            "grid": grid, "block": block, "tile_elems": tile,
            "l2": "fits L2: timed warm (back to back) and cold (512 MB flush between launches)" if fits_l2
                  else "inputs larger than L2 (no flush)",
            "parallelism": f"{args.sharding} x{world}" if world > 1 else "single",
        },
        "clocks": clocks,
        "gpu_launches": args.steps * merger.launches_per_step,
        "roofline": roofline,
    }

    if not args.no_e2e and args.merge in ("avg", "int4"):
        line["e2e"] = e2e_leg(dd, ctx, merger, args, world)
    else:
        line["e2e"] = None
    if parity is not None:
        line["parity"] = parity
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline_leg(merger, args)
    elif rank == 0:
        line["cpu_baseline"] = None

    # ---- one row per other workload and merge kind (N = 1 only) ------------------------------
    if rank == 0 and world == 1:
        rows = []
        todo = wanted_configs(args, args.workload, args.merge)
        if args.scale != 1.0:        # a shrunk run (profiling): only the rows that reuse the resident buffers
            todo = [x for x in todo if x in ("rda", "int4", "push", "broadcast")]
        for name in [x for x in todo if x in ("rda", "int4", "push", "broadcast")]:
            # the other merge kinds of the headline workload, on the buffers that are already resident
            if w.P == 1 and args.merge == "avg" and w.learner_dtype == "bf16":
                if name == "broadcast":
                    rows.append(broadcast_row(dd, ctx, merger, args, ceilings, probes))
                else:
                    rows.append(config_row(dd, ctx, device, args.workload, name, args, ceilings, probes,
                                           traffic_table, merger=merger))
        merger.free()
        merger = None
        for name in [x for x in todo if x not in ("rda", "int4", "push", "broadcast", "tape24")]:
            if name == "rda_dense150m":
                # six participants: the radial-directional merge in its two-launch form
                rows.append(config_row(dd, ctx, device, "dense150m", "rda", args, ceilings, probes, traffic_table))
                continue
            rows.append(config_row(dd, ctx, device, name, "avg", args, ceilings, probes, traffic_table,
                                   resident="participants" if name == "moe4b" else "all"))
        if probes is not None:
            probes.close()
            probes = None
        if "tape24" in todo:
            sub = parse_args(["--workload", "tape24", "--steps", "48", "--warmup", "24"])
            tl = run_replay(sub, ceilings)
            rows.append({"workload": "tape24", "merge": "avg + fused push", "fragments": 24,
                         "params": tl["config"]["model_params"], "M": 8,
                         "ms": {"avg": tl["ms_per_step"]}, "params_per_s": tl["value"],
                         "achieved_gbs": tl["roofline"]["achieved"], "frac": tl["roofline"]["frac"],
                         "frac_of_nominal_8TBs": tl["roofline"]["frac_of_nominal_8TBs"],
                         "write_share": tl["roofline"]["write_share"],
                         "blend_ceiling_gbs": tl["roofline"].get("blend_ceiling_gbs"),
                         "frac_of_blend_ceiling": tl["roofline"].get("frac_of_blend_ceiling"),
                         "steps": 48, "launches_per_merge": 1, "sm_mhz": tl["clocks"]["sm_mhz"],
                         "clock_reasons": tl["clocks"]["reasons"],
                         "note": "one syncer step per bench step: dd_select_quorum + one launch that "
                                 "merges the due fragment and pushes it to the learners that are up; "
                                 "host work included"})
        line["configs"] = rows
    if merger is not None:
        merger.free()
    if probes is not None:
        probes.close()

    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    args = parse_args(argv)
    if args.dry_launch:
        print(json.dumps(launch_plan(max(args.gpus, 1), [a for a in argv if a != "--dry-launch"])), flush=True)
        return 0
    if args.impl == "reference":
        run_reference(args)
        return 0
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args, argv)
    run_ours(args)
    return 0


if __name__ == "__main__":
    sys.exit(main())
