#!/usr/bin/env python
"""Benchmark of the fused per-fragment merge on B200.

One "step" is one pass of the whole hot path -- participation, weights, outer
gradients, weighted reduce, outer optimizer step, norm diagnostics -- over one
synthetic workload (default: one 500M-parameter fragment, 32 bf16 learner
copies of which 24 are in quorum, fp32 global + momentum).  Prints ONE JSON
line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference      # the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "merged_params_per_sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per merged parameter and merge, from the ncu
# captures summarised under profiles/ (absent: not captured for that merge kind and workload).
# The radial-directional figure is the sum of its three passes.
NCU_TRAFFIC_BYTES_PER_PARAM = {
    ("avg", "scale500m"): 63.04, ("avg", "dense150m"): 27.73, ("avg", "dense1b3"): 41.61,
    ("avg", "moe4b"): 41.50, ("rda", "scale500m"): 124.8, ("int4", "scale500m"): 26.24,
}


def host_cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.lower().startswith("model name"):
                    return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="scale500m")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink every fragment (profiling)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-ceilings", action="store_true",
                    help="skip the same-run copy / read bandwidth ceilings (torch kernels)")
    ap.add_argument("--cpu-sample", type=int, default=1 << 27,
                    help="elements of the workload the CPU oracle is timed on")
    ap.add_argument("--out-bf16", action="store_true", help="also write the bf16 broadcast copy")
    ap.add_argument("--unfused-push", action="store_true",
                    help="tape24: separate merge and broadcast launches instead of the fused push")
    ap.add_argument("--merge", choices=["avg", "rda", "int4"], default="avg",
                    help="weighted direct averaging (the headline path), radial-directional, or "
                         "direct averaging of int4-compressed outer gradients")
    ap.add_argument("--resident", choices=["all", "participants"], default="all",
                    help="allocate every learner copy, or only those that take part")
    ap.add_argument("--sharding", choices=["replica", "range"], default="replica",
                    help="N>1: every rank merges its own copy of the workload (weak scaling), or "
                         "each rank owns a contiguous element range of every fragment (strong)")
    return ap.parse_args()


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


# ---- measured peaks -----------------------------------------------------------------

def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measure_ceilings(device, reps=10):
    """What this machine gives plain streaming kernels in the same run (torch library
    kernels, not the product): a device-to-device copy and a read-only reduction."""
    import torch

    n = 1 << 29                                        # 2 GiB of float32 per array
    a = torch.ones(n, dtype=torch.float32, device=device)
    b = torch.empty_like(a)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out = {}
    for name, fn, nbytes in (("copy_ceiling_gbs", lambda: b.copy_(a), 8 * n),
                             ("read_ceiling_gbs", lambda: a.sum(), 4 * n)):
        for _ in range(3):
            fn()
        best = None
        for _ in range(reps):
            ev0.record()
            fn()
            ev1.record()
            ev1.synchronize()
            ms = ev0.elapsed_time(ev1)
            best = ms if best is None or ms < best else best
        out[name] = nbytes / (best * 1e-3) / 1e9
    del a, b
    return out


# ---- the reference arm: the CPU oracle ------------------------------------------------

def run_reference(args):
    """Times the oracle, as it stands, on the host cores: each step is one merge of a
    bounded sample (2^22 elements) of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np

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


def run_replay(args):
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
    merged_params = merged_bytes = launches = 0
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
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes": merged_bytes,
                     "note": ("merge and push fused in one launch per syncer step" if syncer.fused_push else
                              "merge + broadcast launches of the syncer loop") + ", host work included"},
        "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)
    ctx.close()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload == "tape24":
        run_replay(args)
        return

    import numpy as np
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
    frags = build_workload(w, device, rank, args.out_bf16, args.resident)
    ctx = dd.Context(local_rank)
    grid, block, tile = ctx.launch_geometry(dd.BF16 if w.learner_dtype == "bf16" else dd.F32)
    ldtype = dd.BF16 if w.learner_dtype == "bf16" else dd.F32
    records = dd.new_records(w.P, device=device)
    flags = dd.DIAG_STATE
    eta, mu = synth.OUTER_LR, synth.OUTER_MU
    stream = torch.cuda.current_stream()

    int4_codes = int4_scales = None
    if args.merge == "int4":
        # the learners' side, outside the timed region: compress every participant's outer gradient
        assert w.P == 1, "--merge int4 takes a single-fragment workload"
        f = frags[0]
        n0 = f["n"]
        int4_codes, int4_scales = [None] * w.M, [None] * w.M
        for m in range(w.M):
            if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0:
                int4_codes[m] = torch.empty((n0 + 1) // 2, dtype=torch.uint8, device=device)
                int4_scales[m] = torch.empty((n0 + 127) // 128, dtype=torch.float32, device=device)
                ctx.quantize_outer_gradient_int4(f["global_"], f["learners"][m], int4_codes[m],
                                                 int4_scales[m], n=n0, learner_dtype=ldtype)
        torch.cuda.synchronize()

    rda_scratch = None
    if args.merge == "rda" and args.sharding == "range" and world > 1:
        rda_scratch = torch.empty(sum((n + 7) // 8 * 8 for n in w.fragment_sizes), dtype=torch.float32,
                                  device=device)
    # the same buffers are merged every step: marshal their addresses and counts once
    packed_ptrs = dd.pack_pointers(frags[0]["learners"]) if w.P == 1 else None
    packed_tokens = dd.pack_u64(frags[0]["tokens"]) if w.P == 1 else None

    def step(stream=stream):
        if args.merge == "int4":
            f = frags[0]
            ctx.merge_fragment_int4(f["global_"], f["momentum"], int4_codes, int4_scales, f["tokens"],
                                    f["quorum_mask"], f["K"], eta, mu, n=f["n"], flags=flags,
                                    out_bf16=f["out_bf16"], record=records, stream=stream)
        elif args.merge == "rda" and rda_scratch is not None:
            # range-sharded: the passes one by one, norms all-reduced over the ranks in between
            ddist.rda_merge_range_sharded(ctx, frags, w.M, ldtype, eta, mu, records=records,
                                          scratch=rda_scratch, flags=flags, stream=stream)
        elif args.merge == "rda":
            ctx.merge_fragments_batched_rda(frags, w.M, ldtype, eta, mu, flags=flags,
                                            records=records, stream=stream)
        elif w.P == 1:
            f = frags[0]
            ctx.merge_fragment(f["global_"], f["momentum"], packed_ptrs, packed_tokens,
                               f["quorum_mask"], f["K"], eta, mu, n=f["n"], learner_dtype=ldtype,
                               flags=flags, out_bf16=f["out_bf16"], record=records, stream=stream)
        else:
            ctx.merge_fragments_batched(frags, w.M, ldtype, eta, mu, flags=flags, records=records,
                                        stream=stream)

    # ---- parity evidence on the buffers that are about to be timed: sampled windows of
    # the very first merge (fresh state) against the oracle -----------------------------
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and args.merge == "avg":
        import oracle
        f = frags[0]
        n = f["n"]
        win = min(1 << 16, n)
        starts = sorted({0, max(0, (n - win) // 8 * 8), (n // 3) // 8 * 8, (2 * n // 3) // 8 * 8})
        starts = [s0 for s0 in starts if s0 + win <= n]
        part = [m for m in range(w.M) if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0]

        def host_learner(t):
            t = t.cpu()
            return t.view(torch.int16).numpy().view(np.uint16).copy() if t.dtype == torch.bfloat16 \
                else t.numpy().copy()

        saved = [(f["global_"][s0:s0 + win].cpu().numpy().copy(),
                  f["momentum"][s0:s0 + win].cpu().numpy().copy(),
                  [host_learner(f["learners"][m][s0:s0 + win]) if m in part else None
                   for m in range(w.M)]) for s0 in starts]
        step()
        torch.cuda.synchronize()
        rec = dd.read_records(records)[0]
        worst = {"t": 0.0, "v": 0.0}
        exact = True
        for s0, (t0, v0, ls) in zip(starts, saved):
            ref = oracle.merge_fragment(t0, v0, ls, f["tokens"], f["quorum_mask"], f["K"], eta, mu)
            exact &= (rec.status, rec.n_part, rec.idx) == (ref.status, ref.n_part, ref.idx)
            exact &= rec.w_hat == [float(np.float32(x)) for x in ref.w_hat]
            for got, want, which in ((f["global_"], t0, "t"), (f["momentum"], v0, "v")):
                g = got[s0:s0 + win].cpu().numpy().astype(np.float64)
                o = want.astype(np.float64)
                rms = float(np.sqrt(np.mean(o * o))) or 1.0
                worst[which] = max(worst[which], float(np.max(np.abs(g - o) / np.maximum(np.abs(o), rms))))
        parity = {"windows": len(starts), "window_elems": win, "max_err_theta": worst["t"],
                  "max_err_momentum": worst["v"], "tolerance": 1e-5,
                  "participation_and_weights_bit_exact": bool(exact),
                  "metric": "first merge: max |gpu - oracle| / max(|oracle|, rms(oracle))"}

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    recs = dd.read_records(records)
    assert all(r.status == 0 for r in recs), [r.status for r in recs]

    sampler = ClockSampler(local_rank)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    events[0].record(stream)
    for k in range(args.steps):
        step()
        events[k + 1].record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    if world > 1:
        dist.barrier()
    total_ms = events[0].elapsed_time(events[-1])
    per_launch_ms = [events[k].elapsed_time(events[k + 1]) for k in range(args.steps)]
    max_ms = ddist.max_over_ranks(total_ms, device=device)

    # A workload that fits in L2 (126 MB) is also timed cold: a 512 MB buffer is
    # rewritten between launches and only the merge is bracketed by events.
    cold_ms = None
    if w.algorithmic_bytes(out_bf16=args.out_bf16) < 4 * 126e6:
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)
        cold = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for k in range(min(args.steps, 20)):
            flush.fill_(k & 0xff)
            e0.record(stream)
            step()
            e1.record(stream)
            e1.synchronize()
            cold.append(e0.elapsed_time(e1))
        cold_ms = {"median": statistics.median(cold), "min": min(cold), "max": max(cold)}
        del flush

    # A single small fragment is launch-bound from Python (the host needs longer to issue a
    # merge than the GPU to run it): the same calls captured once into a CUDA graph and
    # replayed give the device-bound time per merge.  The library call is capture-safe
    # (one kernel launch, no allocation or synchronisation once the workspace exists).
    graph_ms = None
    if cold_ms is not None and w.P == 1 and args.merge == "avg":
        side = torch.cuda.Stream(device=device)
        graph = torch.cuda.CUDAGraph()
        reps = 50
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for _ in range(reps):
                    step(side)
        torch.cuda.synchronize()
        times = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(8):
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1) / reps)
        graph_ms = {"median": statistics.median(times[3:]), "min": min(times[3:]), "merges_per_graph": reps}
        del graph

    params_per_step = w.total_params
    value = ddist.whole_job_rate(job_params, args.steps, 1, max_ms)
    alg_bytes = w.algorithmic_bytes(out_bf16=args.out_bf16)
    launches_per_step = 1
    if args.merge == "int4":
        alg_bytes = sum(int(n * (w.participants(p) * (0.5 + 4.0 / 128.0) + 16))
                        for p, n in enumerate(w.fragment_sizes))
    if args.merge == "rda":
        # learner copies and Theta are read twice (norms, direction), the direction is
        # written and read back once: 2 (s b + 4) + 24 bytes per parameter
        esz = 2 if w.learner_dtype == "bf16" else 4
        alg_bytes = sum(n * (2 * (w.participants(p) * esz + 4) + 24)
                        for p, n in enumerate(w.fragment_sizes))
        launches_per_step = 3
    avg_launch_ms = sum(per_launch_ms) / len(per_launch_ms)
    slowest = sorted(range(len(per_launch_ms)), key=lambda k: -per_launch_ms[k])[:3]
    achieved = alg_bytes / (avg_launch_ms * 1e-3) / 1e9
    peak, peak_kind = hbm_peak()
    traffic_pp = None if args.out_bf16 else NCU_TRAFFIC_BYTES_PER_PARAM.get((args.merge, args.workload))
    roofline = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": f"of {peak_kind}",
        "traffic": None if traffic_pp is None else traffic_pp * params_per_step,
        "algorithmic_bytes_per_launch": alg_bytes,
        "bytes_per_param": alg_bytes / params_per_step,
        "kernel_ms": {"avg": avg_launch_ms, "median": statistics.median(per_launch_ms),
                      "min": min(per_launch_ms), "max": max(per_launch_ms),
                      "slowest_steps": slowest},
        "frac_of_nominal_8TBs": achieved / 8000.0,
    }
    if graph_ms is not None:
        roofline["ms_per_merge_cuda_graph_replay"] = graph_ms
    if cold_ms is not None:
        roofline["kernel_ms_l2_flushed"] = cold_ms
        roofline["achieved_l2_flushed"] = alg_bytes / (cold_ms["median"] * 1e-3) / 1e9
    if not args.no_ceilings:
        roofline["same_run_ceilings"] = measure_ceilings(device)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": max_ms / args.steps, "higher_is_better": True,
        "scaling": "weak" if args.sharding == "replica" else "strong", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": w.name, "fragments": w.P, "params_per_step": params_per_step, "M": w.M,
            "participants": [w.participants(p) for p in range(w.P)],
            "learner_dtype": w.learner_dtype, "state_dtype": "f32", "outer_lr": eta,
            "outer_mu": mu, "flags": "nesterov+diag_state", "out_bf16": bool(args.out_bf16),
            "merge": args.merge,
            "grid": grid, "block": block, "tile_elems": tile,
            "l2": "inputs larger than L2 (no flush)" if alg_bytes > 4 * 126e6
                  else "fits L2: timed warm (back to back) and cold (512 MB flush between launches)",
            "parallelism": f"{args.sharding} x{world}" if world > 1 else "single",
        },
        "clocks": sampler.summary(),
        "gpu_launches": args.steps * launches_per_step,
        "roofline": roofline,
    }

    # ---- end to end: host buffers through dd_merge_fragment_host -------------------
    if not args.no_e2e and w.P == 1 and args.merge == "avg":
        f = frags[0]
        n = f["n"]
        part = [m for m in range(w.M) if (f["quorum_mask"] >> m) & 1 and f["tokens"][m] > 0]
        # Page-locked host memory is bounded: every rank of the node pins its own buffers, so
        # with several ranks (or little free host memory) the end-to-end leg streams a leading
        # slice of the fragment instead of all of it.
        esz0 = 2 if w.learner_dtype == "bf16" else 4
        per_elem = len(part) * esz0 + 8
        try:
            avail = next(int(l.split()[1]) * 1024 for l in open("/proc/meminfo") if l.startswith("MemAvailable"))
        except Exception:
            avail = 64 << 30
        local_world = int(os.environ.get("LOCAL_WORLD_SIZE", str(world)))
        budget = int(0.4 * avail / max(local_world, 1))
        n = max(8, min(n, budget // per_elem) // 8 * 8)
        h_theta = torch.empty(n, dtype=torch.float32, pin_memory=True)
        h_mom = torch.empty(n, dtype=torch.float32, pin_memory=True)
        h_theta.copy_(f["global_"][:n])
        h_mom.copy_(f["momentum"][:n])
        h_learners = [None] * w.M
        for m in part:
            h_learners[m] = torch.empty(n, dtype=f["learners"][m].dtype, pin_memory=True)
            h_learners[m].copy_(f["learners"][m][:n])
        esz = 2 if w.learner_dtype == "bf16" else 4
        h2d = n * (len(part) * esz + 8)
        d2h = n * 8 + dd.RECORD_BYTES
        ctx.merge_fragment_host(h_theta, h_mom, h_learners, f["tokens"], f["quorum_mask"], f["K"],
                                eta, mu, n=n, learner_dtype=ldtype, flags=flags)      # warm-up
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            rec = ctx.merge_fragment_host(h_theta, h_mom, h_learners, f["tokens"],
                                          f["quorum_mask"], f["K"], eta, mu, n=n,
                                          learner_dtype=ldtype, flags=flags)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        assert rec.status == 0
        dt_max = ddist.max_over_ranks(dt, device=device)
        # every rank streams its own copy (or its own range) of n elements per step
        e2e_params = n * world
        line["e2e"] = {"value": e2e_params * args.e2e_steps / dt_max, "unit": UNIT,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "steps": args.e2e_steps, "elements_per_rank_step": n,
                       "path": "dd_merge_fragment_host: pinned host buffers, chunked H2D -> "
                               "kernel -> D2H pipeline, blocking"}
        del h_learners, h_theta, h_mom
    else:
        line["e2e"] = None

    if parity is not None:
        line["parity"] = parity

    # ---- the oracle on the host cores, bounded sample of the same workload -----------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        f = frags[0]
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
        oracle.merge_fragment(theta, mom, learners, f["tokens"], f["quorum_mask"], f["K"], eta, mu)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": ns / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
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
                                            eta, mu)
            dt_all = time.perf_counter() - t0
            line["cpu_baseline"]["all_cores"] = {"value": ns / dt_all, "unit": UNIT, "cores": cores,
                                                 "kind": "oracle element loop under OpenMP",
                                                 "seconds": dt_all}
        except Exception as exc:      # no OpenMP runtime on the box: the oracle figure stands alone
            line["cpu_baseline"]["all_cores"] = {"unavailable": str(exc)[:120]}
    elif rank == 0:
        line["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
