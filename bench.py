#!/usr/bin/env python
"""Benchmark of the SparseLoCo outer step (metric: outer-step params/s and achieved HBM GB/s).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one whole outer step -- pseudo-gradient, error feedback, chunk-wise Top-k, 2-bit
quantise + pack, error subtract, decode/average of the R payloads, outer update -- for all R
resident workers of the workload, through the C ABI (sl_outer_step).  Prints ONE JSON line.

The path has no exchange between GPUs (R workers are R buffer sets on one GPU), so with N > 1 every
rank runs an independent replica of the workload ("replicas only"): value = N x params / max time.

--impl reference times the CPU oracle (test infrastructure, a deliberately plain program) on a
bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sparseloco_outer_step_params_per_s"
UNIT = "params/s"
DEFAULT_WORKLOAD = "c5_dense_d2048"

# DRAM bytes per ef_select_kernel launch counted by ncu (dram__bytes_read.sum + dram__bytes_write.sum) on one
# decoder layer of the same model, as bytes per (parameter x worker): 13.3264 GB / (67,112,960 x 16).
# Set to None whenever the kernel changes until the counters are taken again.
NCU_EF_SELECT_DRAM_BYTES_PER_PARAM_WORKER = 12.410


def record_stride(k: int) -> int:
    return ((12 * k + 7) // 8 + (2 * k + 7) // 8 + 15) // 16 * 16


def algorithmic_bytes_per_param(R: int, k: int) -> float:
    """Bytes the method must move per parameter per outer step (fp32 state): per worker theta_r
    read + e read + e write; theta_sync read once by the compression and read + written by the
    update; every payload written once and read once."""
    return R * 12 + 4 + 8 + R * 2 * record_stride(k) / 4096.0


def ef_select_bytes_per_param(R: int) -> float:
    return R * 12 + 4


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.2] or [l for (_, l) in self.lines]
        sm, smax, power, reasons = [], [], [], set()
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: the job's time when every rank runs its own replica."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(params: int, steps: int, ms_max: float, world: int) -> float:
    """Whole-job params/s: every rank processed `params` per step in `ms_max` milliseconds."""
    return world * params * steps / (ms_max * 1e-3)


def pick_distinct_locals(torch, wl, k: int, flat: int, payload_bytes: int, workspace_bytes: int) -> int:
    """How many distinct theta_local buffers fit (worker r reads buffer r % D)."""
    free, _total = torch.cuda.mem_get_info()
    fixed = (1 + wl.R) * 4 * flat + wl.R * payload_bytes + workspace_bytes + (6 << 30)
    for D in [wl.R] + [d for d in (32, 16, 8, 4, 2, 1) if d < wl.R]:
        shifted = 0 if D == wl.R else 4 * ALIAS_SHIFT * ((wl.R + D - 1) // D - 1)
        if fixed + D * (4 * flat + shifted) <= free:
            return D
    raise RuntimeError(f"workload {wl.name} does not fit: need {fixed + 4 * flat} bytes, {free} free")


ALIAS_SHIFT = 1 << 26  # elements (268 MB) between the views of two workers that share a theta_local buffer


def make_locals(torch, I, wl, theta, D: int, shift: int):
    """theta_local of every worker when only D < R distinct buffers fit.  Worker r reads buffer r % D
    through a view that starts (r // D) * shift elements into it (the buffers are that much longer,
    the tail filled with noise of theta's scale), so two workers that share a buffer read addresses
    268 MB apart for the same chunk: every one of the R reads of a chunk comes from HBM, as it would
    with R distinct buffers.  With shift = 0 the workers read identical views and the second read of
    a chunk can be served from L2.  Returns (storage, views)."""
    flat = theta.numel()
    extra = shift * ((wl.R + D - 1) // D - 1)
    storage, views = [], []
    for d in range(D):
        buf = torch.empty(flat + extra, dtype=torch.float32, device=theta.device)
        I.theta_local(wl, theta, d, 0, out=buf)
        if extra:
            g = torch.Generator(device=theta.device).manual_seed(77_000 + d)
            buf[flat:].normal_(0.0, 0.02, generator=g)
        storage.append(buf)
    for r in range(wl.R):
        o = (r // D) * shift
        views.append(storage[r % D][o:o + flat])
    return storage, views


def run_ours(args) -> dict:
    import torch
    import torch.distributed as dist
    from paper_2508_15706_b200 import inputs as I
    from paper_2508_15706_b200.binding import SparseLoCo

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the outer step has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = I.workload(args.workload)
    if args.R:
        import dataclasses
        wl = dataclasses.replace(wl, R=args.R)
    k = args.k or wl.k
    shapes = [(t.rows, t.cols) for t in wl.tensors]
    offs = I.offsets(wl.tensors)
    flat = I.flat_numel(wl.tensors)
    N = wl.numel

    sl = SparseLoCo(shapes, offs, k=k, R=wl.R, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr, alloc_workspace=False)
    deferred = args.ef_subtract == "deferred"
    sl.set_ef_deferred(deferred)
    if args.tile_copies != "auto":
        sl.set_tile_copies(args.tile_copies == "tma")
    D = args.distinct_locals or pick_distinct_locals(torch, wl, k, flat, sl.payload_bytes(), sl.workspace_bytes())
    shift = args.alias_shift if D < wl.R else 0
    ws = torch.empty(sl.workspace_bytes(), dtype=torch.uint8, device=dev)
    sl.set_workspace(ws)
    theta = I.theta_sync(wl, dev)
    local, locals_r = make_locals(torch, I, wl, theta, D, shift)
    e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(wl.R)]
    payloads = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(wl.R)]
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()

    for _ in range(args.warmup):
        sl.outer_step(theta, locals_r, e, payloads)
    torch.cuda.synchronize()
    sl.profile_enable(True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        sl.outer_step(theta, locals_r, e, payloads)
    if deferred:  # the subtraction of the last step is still owed: it belongs to the timed work
        sl.ef_flush()
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t0, t1)
    prof = sl.profile_read()
    sl.profile_enable(False)
    ms_max = max_over_ranks(ms, world, dev)
    ms_per_step = ms_max / args.steps
    value = job_value(N, args.steps, ms_max, world)

    # roofline of the dominant kernel, timed live with CUDA events inside the timed region
    top = max(prof.items(), key=lambda kv: kv[1][0])
    ef_ms, ef_n = prof["ef_select"]
    ef_avg_ms = ef_ms / max(ef_n, 1)
    ef_bytes = ef_select_bytes_per_param(wl.R) * N
    peak, peak_src = measured_peak_gbs()
    achieved = ef_bytes / (ef_avg_ms * 1e-3) / 1e9
    traffic = None
    if NCU_EF_SELECT_DRAM_BYTES_PER_PARAM_WORKER is not None:
        traffic = NCU_EF_SELECT_DRAM_BYTES_PER_PARAM_WORKER * N * wl.R
    step_bytes = algorithmic_bytes_per_param(wl.R, k) * N
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    kernel_ms = {name: round(v[0] / max(v[1], 1), 4) for name, v in prof.items()}

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "params": N, "tensors": len(wl.tensors), "R": wl.R, "k": k, "H": wl.H,
                   "chunk": 4096, "beta": wl.beta, "outer_lr": wl.outer_lr,
                   "distinct_theta_local_buffers": D,
                   "theta_local_sharing": ("none" if D == wl.R else
                                           f"worker r reads buffer r % {D} through a view shifted by (r // {D}) x {shift} elements"
                                           if shift else f"worker r reads buffer r % {D} (identical views: L2 can serve re-reads)"),
                   "tile_copies": args.tile_copies,
                   "ef_subtract": args.ef_subtract + (" (each step substitutes the previous step's corrected values "
                                                      "while streaming e; a final flush is inside the timed region)"
                                                      if deferred else ""),
                   "l2": "inputs larger than L2 (every buffer is %.1f GB; state evolves every step)" % (4 * flat / 1e9),
                   "multi_gpu": "replicas only (no data-path collective)"},
        "clocks": clocks,
        "gpu_launches": 8 * args.steps + (1 if deferred else 0),
        "roofline": {"bound": "hbm", "kernel": "ef_select", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": ef_bytes, "avg_launch_ms": ef_avg_ms,
                     "dominant_by_time": top[0]},
        "step_roofline": {"algorithmic_bytes_per_param": algorithmic_bytes_per_param(wl.R, k),
                          "achieved_gbs": step_gbs, "frac_of_measured_peak": step_gbs / peak,
                          "frac_of_nominal_8000": step_gbs / 8000.0},
        "kernel_ms_per_launch": kernel_ms,
    }

    if rank == 0 and world == 1 and not args.no_dense:
        # the paper's dense comparator on the same buffers: DiLoCo's outer step (Eq. 1), R reads of
        # theta_local plus theta and momentum read + written = (4 R + 16) bytes per parameter.
        # (Timed after the headline loop; it borrows one error buffer as the momentum.)
        if deferred:
            sl.ef_flush()
        mom = e[-1]
        mom.zero_()
        for _ in range(2):
            sl.diloco_step(theta, locals_r, mom, 0.9)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        for _ in range(5):
            sl.diloco_step(theta, locals_r, mom, 0.9)
        d1.record(stream)
        torch.cuda.synchronize()
        dms = d0.elapsed_time(d1) / 5
        dbytes = (4 * wl.R + 16) * N
        result["dense_diloco_step"] = {"ms_per_step": dms, "params_per_s": N / (dms * 1e-3),
                                       "achieved_gbs": dbytes / (dms * 1e-3) / 1e9,
                                       "frac_of_measured_peak": dbytes / (dms * 1e-3) / 1e9 / peak,
                                       "entry_point": "sl_diloco_step", "beta_outer": 0.9}
    if rank == 0 and world == 1 and not args.no_dense and deferred:
        # the same step with the error correction written in place by every step (the library's
        # default mode), for comparison with the headline's deferred form
        sl.ef_flush()
        sl.set_ef_deferred(False)
        sl.outer_step(theta, locals_r, e, payloads)
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record(stream)
        for _ in range(5):
            sl.outer_step(theta, locals_r, e, payloads)
        m1.record(stream)
        torch.cuda.synchronize()
        mms = m0.elapsed_time(m1) / 5
        result["materialised_step"] = {"ms_per_step": mms, "params_per_s": N / (mms * 1e-3),
                                       "note": "sl_outer_step with sl_set_ef_deferred(0): e = u - Dhat written by a "
                                               "scattered pass in every step"}
        sl.set_ef_deferred(True)
    if rank == 0 and world == 1 and not args.no_dense:
        # the two halves of the step through their own entry points, one worker per sl_compress call: first with
        # the error correction written in place, then (one worker, called again and again as a rank of the
        # worker-per-GPU deployment does) with it deferred
        if deferred:
            sl.ef_flush()
        sl.set_ef_deferred(False)
        p0, p1, p2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        sl.compress(theta, locals_r[0], e[0], payloads[0])
        p0.record(stream)
        for r in range(wl.R):
            sl.compress(theta, locals_r[r], e[r], payloads[r])
        p1.record(stream)
        for _ in range(3):
            sl.aggregate_apply(payloads, theta)
        p2.record(stream)
        torch.cuda.synchronize()
        cms, ams = p0.elapsed_time(p1) / wl.R, p1.elapsed_time(p2) / 3
        sl.set_ef_deferred(True)
        for _ in range(2):
            sl.compress(theta, locals_r[0], e[0], payloads[0])
        p3, p4 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p3.record(stream)
        for _ in range(8):
            sl.compress(theta, locals_r[0], e[0], payloads[0])
        p4.record(stream)
        sl.ef_flush()
        torch.cuda.synchronize()
        if not deferred:
            sl.set_ef_deferred(False)
        result["parts"] = {
            "sl_compress_deferred_ms_per_worker": p3.elapsed_time(p4) / 8,
            "sl_compress_ms_per_worker": cms,
            "sl_compress_gbs": (16 + 2 * record_stride(k) / 4096.0) * N / (cms * 1e-3) / 1e9,
            "sl_aggregate_apply_ms": ams,
            "sl_aggregate_apply_gbs": (8 + wl.R * record_stride(k) / 4096.0) * N / (ams * 1e-3) / 1e9}
    if rank == 0 and world == 1 and args.codec:
        # entropy-coded index format: one worker's payload of the last step, encode and decode
        coded = torch.empty(sl.coded_payload_capacity(), dtype=torch.uint8, device=dev)
        size = torch.zeros(1, dtype=torch.int64, device=dev)
        back = torch.empty_like(payloads[0])
        for _ in range(3):
            sl.encode_payload(payloads[0], coded, size)
            sl.decode_payload(coded, back)
        c0, c1, c2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        c0.record(stream)
        for _ in range(10):
            sl.encode_payload(payloads[0], coded, size)
        c1.record(stream)
        for _ in range(10):
            sl.decode_payload(coded, back)
        c2.record(stream)
        torch.cuda.synchronize()
        chunks, slots = sl.num_chunks()
        nbytes = int(size.item())
        code_block = (2 * k + 7) // 8
        result["index_codec"] = {
            "payload_bytes": sl.payload_bytes(), "coded_bytes": nbytes, "round_trip_identical": bool(torch.equal(back, payloads[0])),
            "index_bits_per_value": 8.0 * (nbytes - 16 * len(wl.tensors) - code_block * chunks) / slots,
            "encode_ms": c0.elapsed_time(c1) / 10, "decode_ms": c1.elapsed_time(c2) / 10}
        # the update straight from R coded payloads (decoding fused into the update kernel) beside the
        # update from R 12-bit payloads; every worker's slot is given the same coded payload here
        many = [coded] * wl.R
        sl.ef_flush()
        sl.aggregate_apply_coded(many, theta, [nbytes] * wl.R)
        sl.aggregate_apply(payloads, theta)
        c3, c4, c5 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        c3.record(stream)
        for _ in range(3):
            sl.aggregate_apply_coded(many, theta, [nbytes] * wl.R)
        c4.record(stream)
        for _ in range(3):
            sl.aggregate_apply(payloads, theta)
        c5.record(stream)
        torch.cuda.synchronize()
        result["index_codec"]["aggregate_apply_coded_ms"] = c3.elapsed_time(c4) / 3
        result["index_codec"]["aggregate_apply_ms"] = c4.elapsed_time(c5) / 3
        result["index_codec"]["decode_all_workers_then_apply_ms"] = wl.R * result["index_codec"]["decode_ms"] + c4.elapsed_time(c5) / 3
    if rank == 0 and world == 1 and not args.no_e2e:
        del local, locals_r
        torch.cuda.empty_cache()
        result["e2e"] = run_e2e(torch, I, sl, wl, theta, e, payloads, flat, N, args)
    elif not args.no_e2e:
        result["e2e"] = None
    if rank == 0 and world == 1 and not args.no_alias_check and wl.name == DEFAULT_WORKLOAD:
        # everything of the main workload goes before the check allocates its own
        del sl, ws, theta, e, payloads
        local = locals_r = None
        torch.cuda.empty_cache()
        result["theta_local_sharing_check"] = sharing_check(torch, I, dev, peak)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl, k, budget_s=args.cpu_budget)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return result if rank == 0 else None


def time_compression_kernel(torch, sl, theta, locals_r, e, payloads, steps: int = 4) -> float:
    """Average milliseconds of the compression kernel over `steps` outer steps (CUDA events recorded by
    the library around the kernel on the launch stream), after two warm-up steps."""
    for _ in range(2):
        sl.outer_step(theta, locals_r, e, payloads)
    torch.cuda.synchronize()
    sl.profile_enable(True)
    for _ in range(steps):
        sl.outer_step(theta, locals_r, e, payloads)
    torch.cuda.synchronize()
    ms, n = sl.profile_read()["ef_select"]
    sl.profile_enable(False)
    return ms / max(n, 1)


def sharing_check(torch, I, dev, peak: float) -> dict:
    """What sharing theta_local buffers between workers does to the compression kernel's rate.
    (a) half the depth of the 2B config (12 layers), where R = 16 distinct buffers fit: the kernel
        timed with 16 distinct buffers, with 8 buffers read through shifted views (the headline's
        arrangement) and with 8 buffers read through identical views;
    (b) the full 2B config with R = 8 workers and 8 distinct buffers (nothing shared)."""
    from paper_2508_15706_b200.binding import SparseLoCo
    out = {}

    def build(wl):
        shapes = [(t.rows, t.cols) for t in wl.tensors]
        sl = SparseLoCo(shapes, I.offsets(wl.tensors), k=wl.k, R=wl.R, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr,
                        alloc_workspace=False)
        sl.set_ef_deferred(True)
        ws = torch.empty(sl.workspace_bytes(), dtype=torch.uint8, device=dev)
        sl.set_workspace(ws)
        theta = I.theta_sync(wl, dev)
        e = [I.initial_error(wl, r, dev, scale=0.5) for r in range(wl.R)]
        payloads = [torch.zeros(sl.payload_bytes(), dtype=torch.uint8, device=dev) for _ in range(wl.R)]
        return sl, ws, theta, e, payloads

    wl = I.workload("c5_l12")
    N = wl.numel
    sl, ws, theta, e, payloads = build(wl)
    bytes_launch = ef_select_bytes_per_param(wl.R) * N
    storage, views = make_locals(torch, I, wl, theta, wl.R, 0)
    rows = {}
    ms = time_compression_kernel(torch, sl, theta, views, e, payloads)
    rows["16_distinct"] = ms
    # the first 8 buffers again, shared: the extra tail the shifted views need comes from buffer d + 8
    # (any fp32 content of theta's scale serves), so nothing is re-allocated
    shift = ALIAS_SHIFT
    shifted = None
    try:
        storage8, shifted = make_locals(torch, I, wl, theta, 8, shift)
    except torch.cuda.OutOfMemoryError:
        storage8 = None
    if shifted is not None:
        sl.ef_flush()
        rows["8_shared_shifted_views"] = time_compression_kernel(torch, sl, theta, shifted, e, payloads)
        del storage8, shifted
    sl.ef_flush()
    rows["8_shared_identical_views"] = time_compression_kernel(torch, sl, theta, [views[r % 8] for r in range(wl.R)],
                                                               e, payloads)
    out["c5_l12"] = {"params": N, "R": wl.R, "algorithmic_gb_per_launch": bytes_launch / 1e9,
                     "ms": rows, "gbs": {k_: bytes_launch / (v * 1e-3) / 1e9 for k_, v in rows.items()},
                     "frac_of_measured_peak": {k_: bytes_launch / (v * 1e-3) / 1e9 / peak for k_, v in rows.items()}}
    sl.ef_flush()
    del sl, ws, theta, e, payloads, storage, views
    torch.cuda.empty_cache()

    import dataclasses
    out["variants_c5_l12_R8"] = variants_bench(torch, I, dev, build, peak)
    out["options_c5_l12_R8"] = options_bench(torch, I, dev, peak)
    wl = dataclasses.replace(I.workload(DEFAULT_WORKLOAD), R=8)
    N = wl.numel
    sl, ws, theta, e, payloads = build(wl)
    storage, views = make_locals(torch, I, wl, theta, wl.R, 0)
    ms = time_compression_kernel(torch, sl, theta, views, e, payloads)
    b8 = ef_select_bytes_per_param(wl.R) * N
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(torch.cuda.current_stream())
    for _ in range(4):
        sl.outer_step(theta, views, e, payloads)
    sl.ef_flush()
    t1.record(torch.cuda.current_stream())
    torch.cuda.synchronize()
    step_ms = t0.elapsed_time(t1) / 4
    out["c5_dense_d2048_R8_unshared"] = {
        "params": N, "R": 8, "distinct_theta_local_buffers": 8, "compression_kernel_ms": ms,
        "compression_kernel_gbs": b8 / (ms * 1e-3) / 1e9, "frac_of_measured_peak": b8 / (ms * 1e-3) / 1e9 / peak,
        "ms_per_step": step_ms, "params_per_s": N / (step_ms * 1e-3),
        "step_gbs": algorithmic_bytes_per_param(8, wl.k) * N / (step_ms * 1e-3) / 1e9}
    del sl, ws, theta, e, payloads, storage, views
    torch.cuda.empty_cache()
    return out


def variants_bench(torch, I, dev, build, peak: float) -> dict:
    """The paper's Top-k / local-outer-momentum variants (its appendix on DiLoCo variants, Alg. 2-4) on the
    12-layer stack with R = 8 (their per-worker momenta need R more model-sized buffers): ms per step and
    the rate on each step's algorithmic bytes per parameter."""
    import dataclasses
    wl = dataclasses.replace(I.workload("c5_l12"), R=8)
    N, R = wl.numel, 8
    sl, ws, theta, e, payloads = build(wl)
    sl.set_ef_deferred(False)
    local = [I.theta_local(wl, theta, r, 0) for r in range(R)]
    m_r = [I.initial_error(wl, 100 + r, dev, scale=0.3) for r in range(R)]
    mom = I.initial_error(wl, 99, dev, scale=0.3)
    stream = torch.cuda.current_stream()

    def timed(fn, reps=3):
        fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    pay = 2 * 6 * wl.k / 4096.0  # staged (index, value) pairs written and read, per worker and parameter
    rows = {
        "lom_step (Alg. 2)": (lambda: sl.lom_step(theta, local, m_r, 0.9), 12 * R + 8),
        "lom_step sub_k (Alg. 2, Sub-k)": (lambda: sl.lom_step(theta, local, m_r, 0.9, sub_k=True), 16 * R + 8 + R * pay / 2),
        "diloco_topk_step with EF (Alg. 3)": (lambda: sl.diloco_topk_step(theta, local, e, mom, 0.9), 12 * R + 4 + 16 + R * pay),
        "lom_topk_step with EF (Alg. 4)": (lambda: sl.lom_topk_step(theta, local, m_r, e, 0.9), 28 * R + 12 + R * pay),
    }
    out = {"params": N, "R": R, "k": wl.k}
    for name, (fn, bpp) in rows.items():
        ms = timed(fn)
        out[name] = {"ms_per_step": ms, "algorithmic_bytes_per_param": bpp, "gbs": bpp * N / (ms * 1e-3) / 1e9,
                     "frac_of_measured_peak": bpp * N / (ms * 1e-3) / 1e9 / peak}
    del sl, ws, theta, e, payloads, local, m_r, mom
    torch.cuda.empty_cache()
    return out


def measured_peak_gbs():
    """(HBM copy bandwidth in GB/s, where the figure comes from)."""
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    return float(peaks.get("hbm_gbs", 6650.0)), \
        ("measured (MEASURED_PEAKS.json hbm_gbs)" if "hbm_gbs" in peaks else "fallback 6650 GB/s")


def options_bench(torch, I, dev, peak: float, workload: str = "c5_l12", R: int = 8, only: str = "") -> dict:
    """The settings outside the paper's main configuration (quantiser widths of its ablation, no quantiser,
    densities up to half a chunk, bfloat16 storage) on the 12-layer stack with R = 8: ms per outer step and
    the rate on the state the step must stream ((12 R + 8) bytes per parameter in fp32, half in bfloat16:
    theta_r and e read, e written per worker; theta read and written).  These run in plain kernels."""
    import dataclasses
    from paper_2508_15706_b200.binding import SparseLoCo
    base = dataclasses.replace(I.workload(workload), R=R)
    N = base.numel
    shapes, offs = [(t.rows, t.cols) for t in base.tensors], I.offsets(base.tensors)
    stream = torch.cuda.current_stream()
    cases = [("quant_bits=2 k=64 (the tuned path, materialised subtraction)", 2, 64, False),
             ("quant_bits=1 k=64", 1, 64, False), ("quant_bits=3 k=64", 3, 64, False), ("quant_bits=4 k=64", 4, 64, False),
             ("quant_bits=32 k=64 (no quantiser)", 32, 64, False),
             ("quant_bits=2 k=512", 2, 512, False), ("quant_bits=2 k=2048", 2, 2048, False),
             ("bf16 storage, quant_bits=2 k=64", 2, 64, True),
             ("bf16 storage, quant_bits=2 k=64, deferred subtraction (one flush in the timed region)", 2, 64, True),
             ("quant_bits=2 k=64, deferred subtraction (the headline's mode; one flush in the timed region)", 2, 64, False)]
    out = {"workload": workload, "params": N, "R": R}
    cases = [c for c in cases if only in c[0]]
    if all(c[3] for c in cases):
        # bfloat16 cases alone (a workload whose fp32 state would not fit): build the state buffer by buffer
        theta32 = I.theta_sync(base, dev)
        local32 = e32 = None
    else:
        theta32 = I.theta_sync(base, dev)
        local32 = [I.theta_local(base, theta32, r, 0) for r in range(R)]
        e32 = [I.initial_error(base, r, dev, scale=0.5) for r in range(R)]
    for name, bits, k, half in cases:
        sl = SparseLoCo(shapes, offs, k=k, R=R, beta=base.beta, outer_lr=base.outer_lr, quant_bits=bits,
                        bf16_storage=half)
        pay = [torch.zeros(sl.payload_bytes() if bits != 32 else 16, dtype=torch.uint8, device=dev) for _ in range(R)]
        if half and local32 is None:
            theta = theta32.to(torch.bfloat16)
            local = [I.theta_local(base, theta32, r, 0).to(torch.bfloat16) for r in range(R)]
            e = [I.initial_error(base, r, dev, scale=0.5).to(torch.bfloat16) for r in range(R)]
        elif half:
            theta = theta32.to(torch.bfloat16)
            local = [x.to(torch.bfloat16) for x in local32]
            e = [x.to(torch.bfloat16) for x in e32]
        else:
            theta, local, e = theta32.clone(), local32, [x.clone() for x in e32]
        deferred = "deferred" in name
        if deferred:
            sl.set_ef_deferred(True)
        reps = 5 if deferred else 3
        for _ in range(2):
            sl.outer_step(theta, local, e, pay)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            sl.outer_step(theta, local, e, pay)
        if deferred:
            sl.ef_flush()
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        bpp = (12 * R + 8) * (0.5 if half else 1.0)
        out[name] = {"ms_per_step": ms, "state_bytes_per_param": bpp, "gbs": bpp * N / (ms * 1e-3) / 1e9,
                     "frac_of_measured_peak": bpp * N / (ms * 1e-3) / 1e9 / peak}
        del sl, pay, theta, e
        if half:
            del local
        torch.cuda.empty_cache()
    return out


def run_worker_per_gpu(args) -> dict:
    """--mode worker-per-gpu: one worker per rank (R = number of ranks): sl_compress on the rank's own
    theta_local and e, an NCCL all-gather of the payloads into local memory, sl_aggregate_apply on the
    rank's theta replica.  value = params / max-over-ranks step time (every rank updates the same
    params with R = N workers); per-GPU work is fixed as N grows."""
    import torch
    import torch.distributed as dist
    from paper_2508_15706_b200 import inputs as I
    from paper_2508_15706_b200.binding import SparseLoCo
    from paper_2508_15706_b200.worker_step import WorkerStep

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    import dataclasses
    wl = dataclasses.replace(I.workload(args.workload), R=world)
    k = args.k or wl.k
    shapes = [(t.rows, t.cols) for t in wl.tensors]
    sl = SparseLoCo(shapes, I.offsets(wl.tensors), k=k, R=world, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr)
    theta = I.theta_sync(wl, dev)
    local = I.theta_local(wl, theta, rank, 0)
    e = I.initial_error(wl, rank, dev, scale=0.5)
    coded = args.wire == "coded"
    ws = WorkerStep(sl, sl.payload_bytes(), world, rank, dev, coded=coded,
                    coded_capacity=sl.coded_payload_capacity() if coded else 0)
    sl.set_ef_deferred(True)  # this rank's corrected values wait for its next sl_compress; one flush at the end, timed
    for _ in range(args.warmup):
        ws.step(theta, local, e)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        ws.step(theta, local, e)
    sl.ef_flush()
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    if world > 1:
        dist.barrier()
    ms_max = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    clocks = sampler.stop(t0, t1)
    N = wl.numel
    wire = int(ws.exchange.meta[:, 1].max())
    out = {"metric": METRIC, "value": N * args.steps / (ms_max * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": wl.name, "params": N, "R": world, "k": k, "mode": "worker-per-gpu",
                      "exchange": "all-gather of payloads (torch.distributed, NCCL) into local memory",
                      "wire_format": args.wire, "wire_bytes_per_worker": wire, "plain_payload_bytes": sl.payload_bytes(),
                      "l2": "inputs larger than L2"},
           "clocks": clocks, "gpu_launches": (9 + (3 + world if coded else 0)) * args.steps}
    if world > 1:
        dist.destroy_process_group()
    return out if rank == 0 else None


def run_e2e(torch, I, sl, wl, theta, e, payloads, flat, N, args) -> dict:
    """The same step through the host-buffer entry point: every worker's parameters start in pinned
    host memory and cross to the device inside the timed region; the updated theta_sync is read back."""
    dev = theta.device
    n_host = min(2, wl.R)  # distinct pinned host buffers; worker r reads buffer r % n_host
    host = []
    for d in range(n_host):
        h = torch.empty(flat, dtype=torch.float32, pin_memory=True)
        tmp = I.theta_local(wl, theta, d, 1)
        h.copy_(tmp)
        del tmp
        host.append(h)
    theta_host = torch.empty(flat, dtype=torch.float32, pin_memory=True)
    flat4 = (flat + 3) // 4 * 4
    stage = torch.empty(2 * flat4, dtype=torch.float32, device=dev)
    hosts_r = [host[r % n_host] for r in range(wl.R)]
    torch.cuda.synchronize()
    steps = max(1, min(args.e2e_steps, args.steps))
    sl.outer_step_host(theta, hosts_r, stage, e, payloads, theta_host)  # warm-up
    t0 = time.time()
    for _ in range(steps):
        sl.outer_step_host(theta, hosts_r, stage, e, payloads, theta_host)
    torch.cuda.synchronize()
    dt = time.time() - t0
    return {"value": N * steps / dt, "unit": UNIT, "steps": steps, "ms_per_step": dt / steps * 1e3,
            "h2d_bytes_per_step": wl.R * 4 * flat, "d2h_bytes_per_step": 4 * flat,
            "entry_point": "sl_outer_step_host", "distinct_host_buffers": n_host,
            "checksum": float(theta_host[:1024].double().sum())}


# ---------------------------------------------------------------------------------------------
# CPU oracle legs (the only places bench.py touches oracle/)
# ---------------------------------------------------------------------------------------------

def oracle_sample(wl, k, budget_s: float):
    """A bounded sample of the workload for the oracle: tensors of the first layer, as many as fit
    the time budget (calibrated on one small tensor), all R workers, one whole outer step."""
    import numpy as np
    import oracle as O
    from paper_2508_15706_b200 import inputs as I
    cores = os.cpu_count() or 1
    O.set_threads(cores)
    cand = [j for j, t in enumerate(wl.tensors) if t.layer == 0 and t.rows > 1] or list(range(len(wl.tensors)))

    def make(ids, step):
        tensors = [wl.tensors[j] for j in ids]
        sub = I.Workload(wl.name + "_sample", tensors, R=wl.R, k=k, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr,
                         recipe="normal" if wl.recipe == "moe_zero" else wl.recipe, seed=wl.seed)
        if wl.recipe == "outlier_ties":
            sub = wl
        theta = I.theta_sync(sub, "cpu")
        local = [I.theta_local(sub, theta, r, step).numpy() for r in range(wl.R)]
        e = [I.initial_error(sub, r, "cpu", scale=0.5).numpy() for r in range(wl.R)]
        tab = O.Table([(t.rows, t.cols) for t in sub.tensors], I.offsets(sub.tensors))
        cfg = O.Config(k=k, R=wl.R, H=wl.H, beta=wl.beta, outer_lr=wl.outer_lr)
        return cfg, tab, theta.numpy(), local, e, sum(t.numel for t in sub.tensors)

    # calibrate on the smallest candidate
    j0 = min(cand, key=lambda j: wl.tensors[j].numel)
    cfg, tab, th, lo, e, n0 = make([j0], 0)
    t0 = time.time()
    O.outer_step(cfg, tab, th, lo, e)
    rate = n0 / max(time.time() - t0, 1e-6)
    ids, tot = [], 0
    for j in cand:
        if ids and (tot + wl.tensors[j].numel) / rate > budget_s:
            break
        ids.append(j)
        tot += wl.tensors[j].numel
    return make, ids, cores


def cpu_baseline(wl, k, budget_s: float) -> dict:
    import oracle as O
    make, ids, cores = oracle_sample(wl, k, budget_s)
    cfg, tab, th, lo, e, n = make(ids, 0)
    t0 = time.time()
    O.outer_step(cfg, tab, th, lo, e)
    dt = time.time() - t0
    names = ",".join(wl.tensors[j].name for j in ids)
    out = {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
           "sample": f"one outer step, all R={wl.R} workers, tensors [{names}] = {n} params of {wl.numel}"}
    # the same program on one core, on the smallest tensor of the sample (a few seconds)
    j1 = min(ids, key=lambda j: wl.tensors[j].numel)
    cfg, tab, th, lo, e, n1 = make([j1], 0)
    O.set_threads(1)
    t0 = time.time()
    O.outer_step(cfg, tab, th, lo, e)
    dt1 = time.time() - t0
    O.set_threads(cores)
    out["single_thread"] = {"value": n1 / dt1, "seconds": dt1, "sample": f"tensor {wl.tensors[j1].name}, all R={wl.R} workers"}
    return out


def run_reference(args) -> dict:
    from paper_2508_15706_b200 import inputs as I
    import oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    wl = I.workload(args.workload)
    k = args.k or wl.k
    total = args.steps + args.warmup
    make, ids, cores = oracle_sample(wl, k, budget_s=max(1.0, args.reference_budget / max(total, 1)))
    cfg, tab, th, lo, e, n = make(ids, 0)
    for _ in range(args.warmup):
        O.outer_step(cfg, tab, th, lo, e)
    t0 = time.time()
    for _ in range(args.steps):
        O.outer_step(cfg, tab, th, lo, e)
    dt = time.time() - t0
    value = n * args.steps / dt
    names = ",".join(wl.tensors[j].name for j in ids)
    sample = f"each step = one outer step, all R={wl.R} workers, tensors [{names}] = {n} params of {wl.numel}"
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", str(args.gpus))), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "params": wl.numel, "R": wl.R, "k": k, "H": wl.H, "chunk": 4096},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--R", type=int, default=0, help="override the workload's worker count (profiling)")
    ap.add_argument("--ef-subtract", default="deferred", choices=["deferred", "materialised"],
                    help="where e = u - Dhat is applied at the selected positions: in the next step's streaming "
                         "pass (deferred) or by a scattered write in this step (materialised)")
    ap.add_argument("--tile-copies", default="auto", choices=["auto", "tma", "threads"],
                    help="how the compression kernel moves 64x64 blocks: tensor-map block copies (the library's "
                         "default when the table allows) or per-thread 16-byte asynchronous copies")
    ap.add_argument("--distinct-locals", type=int, default=0,
                    help="distinct theta_local buffers (default: as many as fit, at most R)")
    ap.add_argument("--alias-shift", type=int, default=ALIAS_SHIFT,
                    help="element shift between the views of workers sharing a theta_local buffer (0: identical views)")
    ap.add_argument("--no-alias-check", action="store_true",
                    help="skip the measurement of what sharing theta_local buffers does to the kernel's rate")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "worker-per-gpu"],
                    help="replicas: every rank runs the whole R-worker step on its own GPU (the headline); "
                         "worker-per-gpu: one worker per rank, payloads all-gathered (R = number of ranks)")
    ap.add_argument("--wire", default="plain", choices=["plain", "coded"],
                    help="worker-per-gpu: what travels, the 12-bit payload or its entropy-coded form")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense DiLoCo comparator line")
    ap.add_argument("--codec", action="store_true", help="also time the entropy-coded index format on one payload")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--options-only", action="store_true",
                    help="time only the settings outside the main configuration (options_bench) on --options-workload")
    ap.add_argument("--options-workload", default="c5_l12")
    ap.add_argument("--options-workers", type=int, default=8)
    ap.add_argument("--options-filter", default="", help="run only the options cases whose name contains this")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--reference-budget", type=float, default=150.0, help="seconds for the whole reference run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    if args.impl == "reference":
        out = run_reference(args)
    elif args.options_only:  # the settings outside the main configuration alone (small workloads: profiler captures)
        import torch
        from paper_2508_15706_b200 import inputs as I
        torch.cuda.set_device(0)
        out = options_bench(torch, I, torch.device("cuda", 0), measured_peak_gbs()[0],
                            workload=args.options_workload,
                            R=args.options_workers, only=args.options_filter)
    elif args.mode == "worker-per-gpu":
        out = run_worker_per_gpu(args)
    else:
        out = run_ours(args)
    if out is not None:
        print(json.dumps(out))


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this command line, one per GPU,
    with the environment a launcher would set (rendezvous on 127.0.0.1), and pass on what they print
    (rank 0 alone prints the JSON line).  Returns the first non-zero exit code."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + sys.argv, env=env))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


if __name__ == "__main__":
    main()
