#!/usr/bin/env python
"""Benchmark of the tile-major GEMM hot path on B200.

One step = one pass of the whole path over the Llama-3.1-70B-shaped decode workload:
  relayout (row-major -> tile-major, 4 KB blocks of 16 x 128 bf16) of the four projection weights,
  then for M in {1, 8, 32} tokens the tile-major GEMM of every projection (12 GEMMs),
  then the read-amplification count of every (projection, M) tile-major schedule (12 counts, exact integers).
The metric is algorithmic bytes moved per second (TB/s): relayout 2*K*N*2 bytes, GEMM
2*K*N + 2*M*K + 4*M*N bytes.  Beside it: the same GEMMs on row-major weights, the prefill
(M = 4096, TFLOP/s) and Qwen MoE grouped legs, the end-to-end number through tl_gemm_host with
pinned host buffers, and the CPU oracle on a bounded sample.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
N > 1 (under torchrun) runs N independent replicas: the path has no exchange step.
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

import numpy as np
import torch

from paper_2607_04031_b200 import inputs

G, BR, BC = inputs.DEFAULT_G, *inputs.DEFAULT_BLOCK
METRIC = "tile_major_gemm_path_throughput"
UNIT = "TB/s"
WORKLOAD = "llama3.1-70b decode linear layers (qkv, o, gate_up, down; M in {1,8,32}), bf16 tile-major 4KB blocks 16x128"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode GEMM kernel, from the ncu
# capture summarised in profiles/ (None until a capture exists for this kernel version).
NCU_TRAFFIC_RATIO = 171.80 / 168.23          # (dram read + write) / algorithmic bytes, decode qkv M=8 capture
NCU_TRAFFIC_NOTE = ("profiles/gemm_kernel_decode_qkv_m8.md: 168.02 MB read + 3.78 MB written for 168.23 MB algorithmic; "
                    "scaled to the step's average launch by bytes processed (traffic is proportional to the weight bytes)")


def default_cta(M):
    """CTA tile (token rows, weight columns, weight rows per stage) of the library's decode schedule.  The CPU arm
    may not call the CUDA library, so it counts with these; run_ours() checks them against tl_gemm_plan."""
    return (16 if M <= 16 else 32, 256, 64)


def config_dict(world=1):
    return {"workload": WORKLOAD, "G": G, "block": [BR, BC], "parallelism": f"replicas x{world}",
            "l2": "inputs larger than L2: 1.7 GB of weights stream between two uses of the same weight"}


def gemm_bytes(M, N, K):
    return 2 * K * N + 2 * M * K + 4 * M * N


def relayout_bytes(N, K):
    return 2 * K * N * 2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """SM clock, power and throttle reasons read through NVML every few milliseconds by a thread (read-only
    queries); falls back to `nvidia-smi -lms 200` when NVML cannot be loaded.  mark_timed() brackets the timed
    region so that the samples taken inside it can be told from those taken during the other legs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int):
        self.rows = []          # (time, sm MHz, max MHz, watts, set of reasons)
        self.proc = None
        self.index = index
        self.nvml = None
        self.stop_flag = False
        self.t_begin = self.t_end = None
        self.windows = []       # (label, t0, t1) of the legs measured beside the timed step

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(self.index).uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def mark_timed(self, begin: bool):
        if begin:
            self.t_begin = time.perf_counter()
        else:
            self.t_end = time.perf_counter()

    def window(self, label):
        """with sampler.window("leg"): ... records the interval so that stop() can report the leg's own clocks."""
        outer = self

        class _W:
            def __enter__(self_w):
                torch.cuda.synchronize()
                self_w.t0 = time.perf_counter()

            def __exit__(self_w, *exc):
                torch.cuda.synchronize()
                outer.windows.append((label, self_w.t0, time.perf_counter()))
                return False
        return _W()

    def _poll(self):
        n = self.nvml
        mx = n.nvmlDeviceGetMaxClockInfo(self.handle, n.NVML_CLOCK_SM)
        while not self.stop_flag:
            try:
                sm = n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)
                watts = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                mask = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                why = {k for k, bit in self.REASONS.items() if mask & bit}
                self.rows.append((time.perf_counter(), float(sm), float(mx), watts, why))
            except Exception:
                pass
            time.sleep(0.002)

    def _read(self):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.proc.stdout:
            r = [x.strip() for x in line.split(",")]
            try:
                why = {nm for nm, v in zip(names, r[3:7]) if v.lower().startswith("active")}
                self.rows.append((time.perf_counter(), float(r[0]), float(r[1]), float(r[2]), why))
            except (ValueError, IndexError):
                continue

    def stop(self):
        if self.nvml is None and not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no NVML and no nvidia-smi"]}
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
        else:
            time.sleep(0.25)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        rows = list(self.rows)
        inside = [r for r in rows if self.t_begin is not None and self.t_end is not None and self.t_begin <= r[0] <= self.t_end]
        reasons = set()
        for r in rows:
            reasons |= r[4]
        legs = {}
        for label, t0, t1 in self.windows:
            leg = [r for r in rows if t0 <= r[0] <= t1]
            legs[label] = {"sm_mhz": statistics.median(r[1] for r in leg) if leg else None,
                           "sm_mhz_min": min(r[1] for r in leg) if leg else None,
                           "power_w_max": max(r[3] for r in leg) if leg else None, "samples": len(leg),
                           "reasons": sorted(set().union(*[r[4] for r in leg])) if leg else []}
        # sm_mhz describes the timed region only: null when no sample fell inside it (a very short run)
        return {"sm_mhz": statistics.median(r[1] for r in inside) if inside else None,
                "sm_mhz_whole_run": statistics.median(r[1] for r in rows) if rows else None, "legs": legs,
                "sm_max_mhz": max(r[2] for r in rows) if rows else None,
                "power_w_max": max(r[3] for r in rows) if rows else None,
                "samples": len(rows), "samples_in_timed_region": len(inside),
                "sm_mhz_min_in_timed_region": min(r[1] for r in inside) if inside else None,
                "reasons_in_timed_region": sorted(set().union(*[r[4] for r in inside])) if inside else [],
                "reasons": sorted(reasons), "source": "nvml" if self.nvml is not None else "nvidia-smi"}


# ------------------------------------------------------------------ CPU oracle leg

def oracle_sample(step_budget_s: float):
    """Times the oracle, as it stands, on a bounded slab of the same workload: for each of the four projections
    the first n columns of the weight (n a multiple of the memory tile's width, sized so that the whole sample
    takes about step_budget_s), through relayout, the fp64 product for M in (1, 8, 32) and the brute-force
    read-amplification count of the schedule the CUDA kernels run.  Returns a dict."""
    import oracle as tlo
    cores = tlo.num_threads()
    # calibrate the product's rate on a few columns, then size the slabs for the budget
    Kc, n_cal = 8192, 128
    Ac = inputs.bf16_normal((8, Kc), 1.0, seed=900)
    Bc = inputs.bf16_normal((Kc, n_cal), 0.02, seed=901)
    Bc_t = tlo.relayout(inputs.bits(Bc).view(np.uint8), Kc, n_cal, 2, BR, BC, tlo.TO_TILE_MAJOR).view(np.uint16)
    t0 = time.perf_counter()
    tlo.matmul(inputs.bits(Ac), Bc_t, tlo.TILE_MAJOR, BR, BC, 8, n_cal, Kc)
    rate = 8 * n_cal * Kc / (time.perf_counter() - t0)          # MAC/s
    macs_per_col = sum(inputs.LLAMA_DECODE_M) * sum(K for _, K, _ in inputs.LLAMA70B_PROJ)
    n_cols = int(step_budget_s * 0.8 * rate / macs_per_col) // BC * BC
    n_cols = max(BC, min(min(N for _, _, N in inputs.LLAMA70B_PROJ), n_cols))
    data = []
    for i, (name, K, N) in enumerate(inputs.LLAMA70B_PROJ):
        A = {M: inputs.bits(inputs.bf16_normal((M, K), 1.0, seed=910 + 10 * i + M)) for M in inputs.LLAMA_DECODE_M}
        data.append((K, A, inputs.bits(inputs.bf16_normal((K, n_cols), 0.02, seed=902 + i))))
    t0 = time.perf_counter()
    nbytes = 0
    for K, A, Bb in data:
        Bt = tlo.relayout(Bb.view(np.uint8), K, n_cols, 2, BR, BC, tlo.TO_TILE_MAJOR).view(np.uint16)
        for M in inputs.LLAMA_DECODE_M:
            tlo.matmul(A[M], Bt, tlo.TILE_MAJOR, BR, BC, M, n_cols, K)
        for M in inputs.LLAMA_DECODE_M:
            cta = default_cta(M)
            tlo.read_amp(M, n_cols, K, cta[0], cta[1], cta[2], tlo.TILE_MAJOR, G, BR, BC, 2)
        nbytes += relayout_bytes(n_cols, K) + sum(gemm_bytes(M, n_cols, K) for M in inputs.LLAMA_DECODE_M)
    dt = time.perf_counter() - t0
    return {"value": nbytes / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
            "sample": f"all four projections (qkv, o, gate_up, down), the first {n_cols} columns of each weight: oracle "
                      f"relayout + fp64 matmul for M in (1,8,32) + brute-force read-amp count of the kernels' schedules"}


def run_reference(args):
    """--impl reference: the oracle on the host cores, one bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as tlo
    tlo.build()
    per_step = max(0.6, min(20.0, 150.0 / max(1, args.steps + args.warmup)))      # the whole run: about 2.5 minutes
    for _ in range(args.warmup):
        oracle_sample(per_step)
    vals = [oracle_sample(per_step) for _ in range(args.steps)]
    secs = sum(v["seconds"] for v in vals)
    value = statistics.mean(v["value"] for v in vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                         "sample": vals[-1]["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------ replicas (the path does not shard)

def max_over_ranks(ms: float, device, world: int) -> float:
    """The slowest rank's device time; every rank gets the same number."""
    if world <= 1:
        return float(ms)
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, steps: int, step_bytes: int, total_ms: float) -> float:
    """TB/s over all replicas: every rank runs the same step on its own data (weak scaling)."""
    return world * steps * step_bytes / (total_ms * 1e-3) / 1e12


# ------------------------------------------------------------------------ GPU legs

class EventTimer:
    """CUDA-event pairs on the current stream, grouped by label; read after a synchronize."""

    def __init__(self):
        self.pairs = {}

    def time(self, label, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        self.pairs.setdefault(label, []).append((a, b))

    def totals_ms(self):
        return {k: (sum(a.elapsed_time(b) for a, b in v), len(v)) for k, v in self.pairs.items()}


def run_ours(args):
    from paper_2607_04031_b200 import binding as tl
    from paper_2607_04031_b200 import build as tl_build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        tl_build.build()
    if world > 1:
        dist.barrier()
    tl.lib()
    peaks = measured_peaks()
    stream = torch.cuda.current_stream()

    # ---- resident inputs (seeded, synthetic)
    W_row, W_tile, A_dec, C_dec = {}, {}, {}, {}
    for i, (name, K, N) in enumerate(inputs.LLAMA70B_PROJ):
        W_row[name] = inputs.bf16_normal((K, N), 0.02, seed=100 + i + 10 * rank, device=str(dev))
        W_tile[name] = torch.empty_like(W_row[name])
        for M in inputs.LLAMA_DECODE_M:
            A_dec[name, M] = inputs.bf16_normal((M, K), 1.0, seed=200 + 10 * i + M, device=str(dev))
            C_dec[name, M] = torch.empty((M, N), dtype=torch.float32, device=dev)
    read_amp_out = {}
    ra_dev = torch.zeros((len(inputs.LLAMA_DECODE_M) * len(inputs.LLAMA70B_PROJ), 3), dtype=torch.int64, device=dev)
    # The counter is fed the schedule each product really runs: the CTA tile comes from the library's plan query.
    plans = {(name, M): tl.gemm_plan(M, N, K, G, BR, BC) for M in inputs.LLAMA_DECODE_M
             for name, K, N in inputs.LLAMA70B_PROJ}
    for (name, M), pl in plans.items():
        assert pl.cta == default_cta(M), f"bench.default_cta({M}) is stale: the library plans {pl.cta}"
    ra_cfgs = tl.read_amp_cfgs((M, N, K, plans[name, M].cta, tl.LAYOUT_TILE_MAJOR, G, BR, BC, 2)
                               for M in inputs.LLAMA_DECODE_M for name, K, N in inputs.LLAMA70B_PROJ)

    rl_srcs = [W_row[name] for name, _, _ in inputs.LLAMA70B_PROJ]
    rl_dsts = [W_tile[name] for name, _, _ in inputs.LLAMA70B_PROJ]
    rl_shapes = [(K, N) for _, K, N in inputs.LLAMA70B_PROJ]

    def one_step(timer: EventTimer | None):
        # One CUDA-event pair per phase: the launches of a phase run back to back, as they do in a decode loop.
        def phase(label, fn):
            if timer:
                timer.time(label, fn)
            else:
                fn()

        def relayouts():
            # the four weights of the layer in one launch (weight-load time, Section 5.1)
            tl.relayout_batch(rl_srcs, rl_dsts, rl_shapes, 2, G, BR, BC, tl.TO_TILE_MAJOR)

        def gemms():
            for M in inputs.LLAMA_DECODE_M:
                for name, K, N in inputs.LLAMA70B_PROJ:
                    tl.gemm(A_dec[name, M], W_tile[name], C_dec[name, M], M, N, K, G, BR, BC)

        def counters():
            # one launch for the step's 12 schedules, queued behind the GEMMs, no wait: the totals land in device
            # memory and are read after the step
            tl.read_amp_batch(ra_cfgs, ra_dev)

        phase("relayout", relayouts)
        phase("gemm_decode", gemms)
        phase("read_amp", counters)

    step_bytes = sum(relayout_bytes(N, K) for _, K, N in inputs.LLAMA70B_PROJ) + \
        sum(gemm_bytes(M, N, K) for _, K, N in inputs.LLAMA70B_PROJ for M in inputs.LLAMA_DECODE_M)
    gemm_step_bytes = sum(gemm_bytes(M, N, K) for _, K, N in inputs.LLAMA70B_PROJ for M in inputs.LLAMA_DECODE_M)
    # batched relayout, one GEMM launch per product (plus its reduction kernel where the plan is the stream-K cut),
    # one batched counter launch
    launches_per_step = 1 + sum(2 if pl.stream_k and pl.grid > 1 else 1 for pl in plans.values()) + 1

    tl.set_stream(stream)
    for _ in range(max(3, args.warmup)):
        one_step(None)
    tl.device_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    timer = EventTimer()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark_timed(True)
    ev0.record()
    for _ in range(args.steps):
        one_step(timer)
    ev1.record()
    torch.cuda.synchronize()
    sampler.mark_timed(False)
    if world > 1:
        dist.barrier()
    total_ms = ev0.elapsed_time(ev1)
    tl.device_status()
    ra_host = ra_dev.cpu().numpy()
    i = 0
    for M in inputs.LLAMA_DECODE_M:
        for name, K, N in inputs.LLAMA70B_PROJ:
            read_amp_out[name, M] = tuple(int(x) for x in ra_host[i])
            i += 1
    total_ms = max_over_ranks(total_ms, dev, world)
    value = whole_job_value(world, args.steps, step_bytes, total_ms)
    kernel_ms = timer.totals_ms()

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (decode GEMM), live CUDA-event durations inside the timed region
    g_ms, g_n = kernel_ms["gemm_decode"]          # one event pair around the 12 GEMM calls of a step
    r_ms, r_n = kernel_ms["relayout"]
    g_n *= 12
    r_n *= 4
    gemm_gbs = args.steps * gemm_step_bytes / (g_ms * 1e-3) / 1e9
    def schedule_name(p_):
        if p_.stream_k:
            return "stream-K + streamk_reduce_kernel"
        return f"split-K in clusters of {p_.cluster_k}" if p_.cluster_k > 1 else f"whole tiles on {p_.grid} CTAs"
    kernels = sorted({f"gemm_kernel<cta {p_.cta_m}x{p_.cta_n}x{p_.cta_k}, weights on {'N' if p_.weights_on_n else 'M'}, "
                      f"{schedule_name(p_)}>" for p_ in plans.values()})
    roofline = {"bound": "hbm", "kernel": "; ".join(kernels), "achieved": gemm_gbs,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gemm_gbs / peaks["hbm_gbs"],
                "peak_source": f"of {peaks['source']}", "frac_of_nominal_8TBs": gemm_gbs / 8000.0,
                "frac_of_nominal_7p7TBs_hgx": gemm_gbs / 7700.0,
                "traffic": NCU_TRAFFIC_RATIO * gemm_step_bytes / 12, "traffic_note": NCU_TRAFFIC_NOTE,
                "algorithmic_bytes_per_launch_avg": gemm_step_bytes / 12,
                "avg_launch_us": g_ms / g_n * 1e3,
                "timing": "CUDA events around the 12 back-to-back GEMM calls of every step; duration per call = phase time / 12"}
    relayout_gbs = args.steps * sum(relayout_bytes(N, K) for _, K, N in inputs.LLAMA70B_PROJ) / (r_ms * 1e-3) / 1e9

    extra = {}
    # ---- per-shape decode table, tile-major next to row-major through the same kernel (cold L2: weights rotate)
    def time_calls(calls, reps):
        for c in calls:
            c()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for c in calls:
                c()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    per_shape = []
    with sampler.window("decode_per_shape"):
        for M in inputs.LLAMA_DECODE_M:
            # one pass over all four weights of a layout, then the other layout, alternating: 1.7 GB between two
            # uses of the same weight, and both layouts under the same clocks
            evs = []
            for rep in range(7):
                for layout in ("tile", "row"):
                    for name, K, N in inputs.LLAMA70B_PROJ:
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record()
                        if layout == "tile":
                            tl.gemm(A_dec[name, M], W_tile[name], C_dec[name, M], M, N, K, G, BR, BC)
                        else:
                            tl.gemm(A_dec[name, M], W_row[name], C_dec[name, M], M, N, K, 0, 0, 0)
                        b.record()
                        if rep > 0:
                            evs.append((name, layout, a, b))
            torch.cuda.synchronize()
            for layout in ("tile", "row"):
                for name, K, N in inputs.LLAMA70B_PROJ:
                    ts = [a.elapsed_time(b) for (n_, l_, a, b) in evs if n_ == name and l_ == layout]
                    med = statistics.median(ts)
                    per_shape.append({"proj": name, "M": M, "layout": layout, "us": med * 1e3,
                                      "GBps": gemm_bytes(M, N, K) / (med * 1e-3) / 1e9})
    extra["decode_per_shape"] = per_shape
    tile_t = sum(x["us"] for x in per_shape if x["layout"] == "tile")
    row_t = sum(x["us"] for x in per_shape if x["layout"] == "row")
    extra["tile_vs_row_time_ratio_decode"] = tile_t / row_t

    # ---- between decode and prefill: the same four weights at 128 and 256 token rows (one launch per event pair; the
    # four weights rotate, 1.7 GB between two uses of the same one)
    mid = []
    with sampler.window("mid_batch"):
        for M in (128, 256):
            A_mid = {K: inputs.bf16_normal((M, K), 1.0, seed=700 + M + K // 1024, device=str(dev))
                     for K in sorted({K for _, K, _ in inputs.LLAMA70B_PROJ})}
            C_mid = {N: torch.empty((M, N), dtype=torch.float32, device=dev) for N in sorted({N for _, _, N in inputs.LLAMA70B_PROJ})}
            evs = {name: [] for name, _, _ in inputs.LLAMA70B_PROJ}
            for rep_ in range(6):
                for name, K, N in inputs.LLAMA70B_PROJ:
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    tl.gemm(A_mid[K], W_tile[name], C_mid[N], M, N, K, G, BR, BC)
                    b.record()
                    if rep_ > 0:
                        evs[name].append((a, b))
            torch.cuda.synchronize()
            for name, K, N in inputs.LLAMA70B_PROJ:
                med = statistics.median(a.elapsed_time(b) for a, b in evs[name])
                pl = tl.gemm_plan(M, N, K, G, BR, BC)
                mid.append({"proj": name, "M": M, "us": med * 1e3, "GBps": gemm_bytes(M, N, K) / (med * 1e-3) / 1e9,
                            "TFLOPs": 2.0 * M * N * K / (med * 1e-3) / 1e12, "cta": list(pl.cta),
                            "schedule": "stream-K" if pl.stream_k else f"clusters of {pl.cluster_k}" if pl.cluster_k > 1
                            else f"whole tiles on {pl.grid} CTAs"})
            del A_mid, C_mid
    extra["llama_mid_batch"] = mid
    tl.device_status()

    # ---- the twelve products captured once into a CUDA graph and replayed, next to the same calls issued directly
    # (alternating, so that both see the same clocks).  The kernels and their programmatic dependencies are the same;
    # what a replay saves is the host's launch work between them.
    with sampler.window("decode_cuda_graph"):
        try:
            def gemms12():
                for M in inputs.LLAMA_DECODE_M:
                    for name, K, N in inputs.LLAMA70B_PROJ:
                        tl.gemm(A_dec[name, M], W_tile[name], C_dec[name, M], M, N, K, G, BR, BC)

            gemms12()
            torch.cuda.synchronize()
            graph12 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph12):
                gemms12()
            evs = {"direct": [], "graph": []}
            for rep_ in range(21):
                for kind, fn in (("direct", gemms12), ("graph", graph12.replay)):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    fn()
                    b.record()
                    if rep_ > 0:
                        evs[kind].append((a, b))
            torch.cuda.synchronize()
            tl.device_status()
            med = {k: statistics.median(a.elapsed_time(b) for a, b in v) for k, v in evs.items()}
            extra["decode_cuda_graph"] = {"direct_us": med["direct"] * 1e3, "graph_us": med["graph"] * 1e3,
                                          "graph_GBps": gemm_step_bytes / (med["graph"] * 1e-3) / 1e9,
                                          "note": "the step's 12 decode products back to back: direct calls and one replayed graph"}
            del graph12
        except Exception as exc:  # report, never hide
            extra["decode_cuda_graph"] = {"error": f"{type(exc).__name__}: {exc}"}

    # ---- the same twelve products as three independent decode batches on three streams (one per batch size, own
    # split-K workspace each): CTAs of one product fill the SMs that the tail of another leaves free.  Reported
    # beside the step, not as the step: inside one decode loop the products depend on each other.
    try:
        ws3 = {M: torch.empty(max(tl.gemm_workspace_bytes(M, N, K) for _, K, N in inputs.LLAMA70B_PROJ) + 256,
                              dtype=torch.uint8, device=dev) for M in inputs.LLAMA_DECODE_M}
        side = {M: torch.cuda.Stream(device=dev) for M in inputs.LLAMA_DECODE_M}
        main_stream = torch.cuda.current_stream()

        def three_streams():
            fork = torch.cuda.Event()
            fork.record(main_stream)
            for M in inputs.LLAMA_DECODE_M:
                side[M].wait_event(fork)
                tl.set_workspace(ws3[M])             # the pointer travels with each launch
                for name, K, N in inputs.LLAMA70B_PROJ:
                    tl.gemm(A_dec[name, M], W_tile[name], C_dec[name, M], M, N, K, G, BR, BC, stream=side[M])
                join = torch.cuda.Event()
                join.record(side[M])
                main_stream.wait_event(join)

        ms3 = time_calls([three_streams], 20)
        tl.set_workspace(None)
        extra["decode_three_streams"] = {"us": ms3 * 1e3, "GBps": gemm_step_bytes / (ms3 * 1e-3) / 1e9,
                                         "note": "12 decode products, one stream per batch size (M = 1, 8, 32)"}
        del ws3
    except Exception as exc:  # report, never hide
        tl.set_workspace(None)
        extra["decode_three_streams"] = {"error": f"{type(exc).__name__}: {exc}"}
    tl.device_status()

    # ---- K-contiguous flavour (weights kept [N][K]; Eq. 2 as printed with the (64, 32) memory tile), M = 8
    W_nk, W_nk_tile = {}, {}
    for name, K, N in inputs.LLAMA70B_PROJ:
        W_nk[name] = W_row[name].t().contiguous()
        W_nk_tile[name] = torch.empty_like(W_nk[name])
        tl.relayout(W_nk[name], W_nk_tile[name], N, K, 2, G, 32, 64, tl.TO_TILE_MAJOR)
    kcont = []
    for layout in ("tile_major_k_32x64", "plain_NK"):
        evs = []
        for rep in range(6):
            for name, K, N in inputs.LLAMA70B_PROJ:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                if layout == "plain_NK":
                    tl.gemm_kmajor(A_dec[name, 8], W_nk[name], C_dec[name, 8], 8, N, K, 0, 0, 0)
                else:
                    tl.gemm_kmajor(A_dec[name, 8], W_nk_tile[name], C_dec[name, 8], 8, N, K, G, 32, 64)
                b.record()
                if rep > 0:
                    evs.append((name, a, b))
        torch.cuda.synchronize()
        for name, K, N in inputs.LLAMA70B_PROJ:
            med = statistics.median(a.elapsed_time(b) for (n_, a, b) in evs if n_ == name)
            kcont.append({"proj": name, "M": 8, "layout": layout, "us": med * 1e3,
                          "GBps": gemm_bytes(8, N, K) / (med * 1e-3) / 1e9})
    extra["k_contiguous_decode_m8"] = kcont
    # FP8 (E4M3) on the same shapes: 4 KB memory tiles of 32 x 128 bytes (and the 64 x 64 tile of Figure 1(c))
    fp8 = []
    A8 = {name: inputs.fp8_normal((8, K), 1.0, seed=700 + i, device=str(dev)).view(torch.uint8)
          for i, (name, K, N) in enumerate(inputs.LLAMA70B_PROJ)}
    for tn, tk in ((32, 128), (64, 64)):
        W8 = {}
        for i, (name, K, N) in enumerate(inputs.LLAMA70B_PROJ):
            w = inputs.fp8_normal((N, K), 0.05, seed=710 + i, device=str(dev)).view(torch.uint8)
            W8[name] = torch.empty_like(w)
            tl.relayout(w, W8[name], N, K, 1, G, tn, tk, tl.TO_TILE_MAJOR)
            del w
        evs = []
        for rep in range(6):
            for name, K, N in inputs.LLAMA70B_PROJ:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                tl.gemm_fp8_kmajor(A8[name], W8[name], C_dec[name, 8], 8, N, K, G, tn, tk)
                b.record()
                if rep > 0:
                    evs.append((name, a, b))
        torch.cuda.synchronize()
        for name, K, N in inputs.LLAMA70B_PROJ:
            med = statistics.median(a.elapsed_time(b) for (n_, a, b) in evs if n_ == name)
            fp8.append({"proj": name, "M": 8, "tile": [tn, tk], "us": med * 1e3,
                        "GBps": (K * N + 8 * K + 4 * 8 * N) / (med * 1e-3) / 1e9})
        del W8
    extra["fp8_decode_m8"] = fp8
    del W_nk, W_nk_tile
    tl.device_status()

    # ---- tile-major aware box loads (Section 4.3, emulated): every 64 x 256 weight-tile load of the gate_up weight
    # kept [N][K] in (64, 32) memory tiles, through a 2-D and through a 4-D view of the same matrix
    name, K, N = inputs.LLAMA70B_PROJ[2]
    w_nk = W_row[name].t().contiguous()
    w_nk_tile = torch.empty_like(w_nk)
    tl.relayout(w_nk, w_nk_tile, N, K, 2, G, 32, 64, tl.TO_TILE_MAJOR)
    del w_nk
    hw = []
    boxes_dst = torch.empty((K // 64) * (N // 256) * 64 * 256, dtype=torch.bfloat16, device=dev)
    c2 = torch.tensor([[i, j] for j in range(0, N, 256) for i in range(0, K, 64)], dtype=torch.int32, device=dev)
    c4 = torch.tensor([[0, 0, i // 64, j // 256] for j in range(0, N, 256) for i in range(0, K, 64)], dtype=torch.int32,
                      device=dev)
    for label, desc, cd in (("2d", tl.hw_desc([K, N], [1, K], [64, 256], 2, 64, 32, K), c2),
                            ("4d", tl.hw_desc([64, 256, K // 64, N // 256], [1, K, 64, 256 * K], [64, 256, 1, 1], 2, 64, 32, K), c4)):
        ms = time_calls([lambda: tl.hw_box_load(desc, w_nk_tile, cd, boxes_dst)], 5)
        hw.append({"view": label, "boxes": int(cd.shape[0]), "ms": ms, "GBps": 2 * 2.0 * K * N / (ms * 1e-3) / 1e9})
    extra["hw_box_load_gate_up"] = hw
    del w_nk_tile, boxes_dst
    tl.device_status()

    # ---- Qwen-3-30B-A3B MoE grouped leg
    q = inputs.QWEN_MOE
    offsets, counts, _ = inputs.zipf_topk_routing(q["tokens"], q["experts"], q["topk"], q["zipf_alpha"], seed=0)
    rows = int(offsets[-1])
    d_off = torch.from_numpy(offsets).to(dev)
    active = int((counts > 0).sum())
    moe = []
    moe_window = sampler.window("qwen_moe")
    moe_window.__enter__()
    for name, K, N in inputs.QWEN_MOE_PROJ:
        # two copies of the expert weights so that consecutive launches do not hit L2 (403-805 MB each anyway)
        Bm = inputs.bf16_normal((q["experts"], K, N), 0.02, seed=400, device=str(dev))
        Bt = torch.empty_like(Bm)
        tl.relayout(Bm, Bt, q["experts"] * K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
        Am = inputs.bf16_normal((rows, K), 1.0, seed=401, device=str(dev))
        Cm = torch.empty((rows, N), dtype=torch.float32, device=dev)
        for layout, buf, blk in (("tile", Bt, (BR, BC)), ("row", Bm, (0, 0))):
            ms = time_calls([lambda: tl.gemm_grouped(Am, buf, Cm, d_off, q["experts"], rows, N, K, G, blk[0], blk[1])], 10)
            nbytes = active * 2 * K * N + 2 * rows * K + 4 * rows * N
            moe.append({"proj": name, "layout": layout, "us": ms * 1e3, "GBps": nbytes / (ms * 1e-3) / 1e9,
                        "active_experts": active})
        ra_t = tl.read_amp_grouped(offsets, N, K, (256, 256, 128), tl.LAYOUT_TILE_MAJOR, G, 32, 64, 2)
        ra_r = tl.read_amp_grouped(offsets, N, K, (256, 256, 128), tl.LAYOUT_ROW_MAJOR, G, 0, 0, 2)
        # ... and of the schedule the grouped kernel runs (its own CTA tile, from the plan query)
        gcta = tl.gemm_plan(rows, N, K, G, BR, BC, (0, 0, 0), q["experts"]).cta
        ka_t = tl.read_amp_grouped(offsets, N, K, gcta, tl.LAYOUT_TILE_MAJOR, G, BR, BC, 2)
        ka_r = tl.read_amp_grouped(offsets, N, K, gcta, tl.LAYOUT_ROW_MAJOR, G, 0, 0, 2)
        moe.append({"proj": name, "read_amp_128x256_weight_tile": {"tile_major_32x64": ra_t[0] / ra_t[1],
                                                                  "row_major": ra_r[0] / ra_r[1]},
                    "read_amp_kernel_schedule": {"cta": list(gcta), "tile_major_16x128": ka_t[0] / ka_t[1],
                                                 "row_major": ka_r[0] / ka_r[1]}})
        del Bm, Bt, Am, Cm
    # the whole expert FFN in one call: gate_up with the gated epilogue (bf16 h) -> down
    hid, inter = q["hidden"], q["inter"]
    Wgu = inputs.bf16_normal((q["experts"], hid, 2 * inter), 0.02, seed=410, device=str(dev))
    Wdn = inputs.bf16_normal((q["experts"], inter, hid), 0.02, seed=411, device=str(dev))
    Wgu_t, Wdn_t = torch.empty_like(Wgu), torch.empty_like(Wdn)
    tl.relayout(Wgu, Wgu_t, q["experts"] * hid, 2 * inter, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    tl.relayout(Wdn, Wdn_t, q["experts"] * inter, hid, 2, G, BR, BC, tl.TO_TILE_MAJOR)
    del Wgu, Wdn
    Xm = inputs.bf16_normal((rows, hid), 1.0, seed=412, device=str(dev))
    Hm = torch.empty((rows, inter), dtype=torch.bfloat16, device=dev)
    Ym = torch.empty((rows, hid), dtype=torch.float32, device=dev)
    ms = time_calls([lambda: tl.moe_ffn(Xm, Wgu_t, Wdn_t, Hm, Ym, d_off, q["experts"], rows, hid, inter, G, BR, BC)], 10)
    ffn_bytes = active * 2 * (hid * 2 * inter + inter * hid) + 2 * rows * hid + 2 * 2 * rows * inter + 4 * rows * hid
    moe.append({"proj": "expert_ffn_chain", "layout": "tile", "us": ms * 1e3, "GBps": ffn_bytes / (ms * 1e-3) / 1e9,
                "active_experts": active, "note": "tl_moe_ffn: grouped gate_up + silu*mul epilogue -> bf16 h -> grouped down"})
    del Xm, Hm, Ym
    # the same expert FFN with more tokens routed the same way (64 and 256 rows per expert on average): the grouped
    # tile grows with the rows per expert
    for tokens_big in (1024, 4096):
        off_b, cnt_b, _ = inputs.zipf_topk_routing(tokens_big, q["experts"], q["topk"], q["zipf_alpha"], seed=0)
        rows_b, act_b = int(off_b[-1]), int((cnt_b > 0).sum())
        d_off_b = torch.from_numpy(off_b).to(dev)
        Xb = inputs.bf16_normal((rows_b, hid), 1.0, seed=413, device=str(dev))
        Hb = torch.empty((rows_b, inter), dtype=torch.bfloat16, device=dev)
        Yb = torch.empty((rows_b, hid), dtype=torch.float32, device=dev)
        ms = time_calls([lambda: tl.moe_ffn(Xb, Wgu_t, Wdn_t, Hb, Yb, d_off_b, q["experts"], rows_b, hid, inter, G, BR, BC)], 6)
        fl = 2.0 * rows_b * (hid * 2 * inter + inter * hid)
        by = act_b * 2 * (hid * 2 * inter + inter * hid) + 2 * rows_b * hid + 2 * 2 * rows_b * inter + 4 * rows_b * hid
        moe.append({"proj": "expert_ffn_chain", "tokens": tokens_big, "rows": rows_b, "layout": "tile", "us": ms * 1e3,
                    "GBps": by / (ms * 1e-3) / 1e9, "TFLOPs": fl / (ms * 1e-3) / 1e12, "active_experts": act_b,
                    "cta": list(tl.gemm_plan(rows_b, 2 * inter, hid, G, BR, BC, (0, 0, 0), q["experts"]).cta)})
        del Xb, Hb, Yb, d_off_b
    del Wgu_t, Wdn_t
    moe_window.__exit__(None, None, None)
    extra["qwen_moe"] = moe
    tl.device_status()

    # ---- Qwen-3-30B-A3B attention projections at M = 256 (dense, tile-major and row-major alternating; weights rotate
    # over enough copies that every launch is L2-cold)
    qattn = []
    with sampler.window("qwen_attention"):
        for name, K, N in inputs.QWEN_ATTN_PROJ:
            copies = max(3, int(300e6 // (2 * K * N)) + 1)
            Wr = [inputs.bf16_normal((K, N), 0.02, seed=500 + c, device=str(dev)) for c in range(copies)]
            Wt = [torch.empty_like(w) for w in Wr]
            for c in range(copies):
                tl.relayout(Wr[c], Wt[c], K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
            Aq = inputs.bf16_normal((256, K), 1.0, seed=520, device=str(dev))
            Cq = torch.empty((256, N), dtype=torch.float32, device=dev)
            evs = {"tile": [], "row": []}
            for rep_ in range(6):
                for c in range(copies):
                    for layout in ("tile", "row"):
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record()
                        if layout == "tile":
                            tl.gemm(Aq, Wt[c], Cq, 256, N, K, G, BR, BC)
                        else:
                            tl.gemm(Aq, Wr[c], Cq, 256, N, K, 0, 0, 0)
                        b.record()
                        if rep_ > 0:
                            evs[layout].append((a, b))
            torch.cuda.synchronize()
            # the same launches back to back without an event between them, direct and as one replayed CUDA graph
            def chain_():
                for c in range(copies):
                    tl.gemm(Aq, Wt[c], Cq, 256, N, K, G, BR, BC)
            chain_us = {}
            try:
                graph_q = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph_q):
                    chain_()
                for kind, fn in (("direct", chain_), ("graph", graph_q.replay)):
                    chain_us[kind] = time_calls([fn], 8) * 1e3 / copies
                del graph_q
            except Exception as exc:  # report, never hide
                chain_us = {"error": f"{type(exc).__name__}: {exc}"}
            for layout in ("tile", "row"):
                med = statistics.median(a.elapsed_time(b) for a, b in evs[layout])
                qattn.append({"proj": name, "M": 256, "layout": layout, "us": med * 1e3,
                              **({"back_to_back_us": chain_us} if layout == "tile" else {}),
                              "GBps": gemm_bytes(256, N, K) / (med * 1e-3) / 1e9,
                              "TFLOPs": 2.0 * 256 * N * K / (med * 1e-3) / 1e12,
                              "cta": list(tl.gemm_plan(256, N, K, G, BR, BC).cta)})
            del Wr, Wt, Aq, Cq
    extra["qwen_attention_m256"] = qattn
    tl.device_status()

    # (The prefill leg comes after every bandwidth-bound leg: it holds the board at its power cap, and the SM clock
    # stays low for a while afterwards, which the clock-sensitive kernels would otherwise be charged with.)
    # ---- prefill leg (M = 4096): tensor-core bound
    Mp = inputs.LLAMA_PREFILL_M
    prefill = []
    # Tile-major and row-major launches alternate (tile, row, tile, row, ... per shape), so that both layouts see the
    # same clocks: a leg that runs second under the power cap would otherwise be charged with the lower clock.
    with sampler.window("prefill"):
        for name, K, N in inputs.LLAMA70B_PROJ:
            Ap = inputs.bf16_normal((Mp, K), 1.0, seed=300, device=str(dev))
            Cp = torch.empty((Mp, N), dtype=torch.float32, device=dev)
            calls = {"tile": lambda: tl.gemm(Ap, W_tile[name], Cp, Mp, N, K, G, BR, BC),
                     "row": lambda: tl.gemm(Ap, W_row[name], Cp, Mp, N, K, 0, 0, 0)}
            for c in calls.values():
                c()
            torch.cuda.synchronize()
            evs = {"tile": [], "row": []}
            for rep_ in range(5):
                for layout in ("tile", "row"):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    calls[layout]()
                    b.record()
                    evs[layout].append((a, b))
            torch.cuda.synchronize()
            for layout in ("tile", "row"):
                ms = statistics.mean(a.elapsed_time(b) for a, b in evs[layout])
                prefill.append({"proj": name, "layout": layout, "ms": ms, "TFLOPs": 2.0 * Mp * N * K / (ms * 1e-3) / 1e12})
            del Ap, Cp
    pt = [x for x in prefill if x["layout"] == "tile"]
    flops = sum(2.0 * Mp * N * K for _, K, N in inputs.LLAMA70B_PROJ)
    tf = flops / (sum(x["ms"] for x in pt) * 1e-3) / 1e12
    pplan = tl.gemm_plan(Mp, 8192, 8192, G, BR, BC)
    extra["prefill"] = {"per_shape": prefill, "TFLOPs_tile_major": tf, "order": "tile, row alternating per launch",
                        "plan_o": pplan.as_dict(),
                        "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                     "frac": tf / peaks["bf16_tflops"], "peak_source": f"of {peaks['source']} (burst)",
                                     "frac_of_nominal_2250": tf / 2250.0},
                        "tile_vs_row_time_ratio": sum(x["ms"] for x in pt) /
                        sum(x["ms"] for x in prefill if x["layout"] == "row")}
    tl.device_status()

    # FP8 (E4M3) prefill on the K-contiguous flavour, 64 x 64 memory tiles: the o and gate_up shapes
    fp8_prefill = []
    for i, (name, K, N) in enumerate(inputs.LLAMA70B_PROJ):
        if name not in ("o", "gate_up"):
            continue
        w8 = inputs.fp8_normal((N, K), 0.05, seed=720 + i, device=str(dev)).view(torch.uint8)
        w8t = torch.empty_like(w8)
        tl.relayout(w8, w8t, N, K, 1, G, 64, 64, tl.TO_TILE_MAJOR)
        del w8
        a8 = inputs.fp8_normal((Mp, K), 1.0, seed=730 + i, device=str(dev)).view(torch.uint8)
        c8 = torch.empty((Mp, N), dtype=torch.float32, device=dev)
        ms = time_calls([lambda: tl.gemm_fp8_kmajor(a8, w8t, c8, Mp, N, K, G, 64, 64)], 5)
        fp8_prefill.append({"proj": name, "tile": [64, 64], "ms": ms, "TFLOPs": 2.0 * Mp * N * K / (ms * 1e-3) / 1e12})
        del w8t, a8, c8
    extra["fp8_prefill"] = {"per_shape": fp8_prefill,
                            "peak_note": "nominal dense FP8 peak 4500 TFLOP/s; 2 x the measured bf16 burst peak = "
                                         f"{2 * peaks['bf16_tflops']:.0f}"}
    tl.device_status()

    # ---- modelled read amplification at 4 KB (exact integers from the counter)
    ra = {}
    shapes = {name: (K, N) for name, K, N in inputs.LLAMA70B_PROJ}
    for (name, M), t_ in read_amp_out.items():
        K, N = shapes[name]
        # the row-major factor of the schedule the same kernel runs on row-major weights (counted outside the timed step)
        row_cta = tl.gemm_plan(M, N, K, 0, 0, 0).cta
        r_ = tl.read_amp(M, N, K, row_cta, tl.LAYOUT_ROW_MAJOR, G, 0, 0, 2)
        ra[f"{name}_M{M}"] = {"tile_major": t_[0] / t_[1], "row_major": r_[0] / r_[1], "cta": list(plans[name, M].cta),
                              "cta_row_major": list(row_cta),
                              "fetched_tile": t_[0], "used": t_[1], "fetched_row": r_[0]}
    extra["read_amp_4KB"] = ra
    # requests shared between the 148 co-resident CTAs of a wave (prefill tiles 256 x 256 x 64, gate_up), and the
    # prefetch degree of Eq. 6 that the per-tile request counts imply on the paper's 4.9 TB/s, 5 us device
    name, K, N = inputs.LLAMA70B_PROJ[2]
    shared = {}
    for label, lt, blk in (("row_major", tl.LAYOUT_ROW_MAJOR, (0, 0)), ("tile_major", tl.LAYOUT_TILE_MAJOR, (BR, BC))):
        plain = tl.read_amp(Mp, N, K, (256, 256, 64), lt, G, blk[0], blk[1], 2)
        sh = tl.read_amp_shared(Mp, N, K, (256, 256, 64), 148, lt, G, blk[0], blk[1], 2)
        loads = (-(-Mp // 256)) * (N // 256) * (K // 64)
        p_tile = max(1, plain[2] // loads)
        shared[label] = {"unshared": plain[0] / plain[1], "shared_by_wave_of_148": sh[0] / sh[1],
                         "requests_per_tile": p_tile,
                         "prefetch_degree_eq6": tl.prefetch_degree(4.9e12, 5e-6, G, 148, 1, p_tile, K, 64, 1.0)}
    extra["read_amp_shared_prefill_gate_up"] = shared

    clocks = sampler.stop()

    # ---- end to end: host buffers through tl_gemm_host (H2D of A and the row-major weight, relayout, GEMM, D2H of C)
    e2e = None
    try:
        scratch = torch.empty(max(tl.gemm_host_scratch_bytes(32, N, K) for _, K, N in inputs.LLAMA70B_PROJ),
                              dtype=torch.uint8, device=dev)
        hW = {name: W_row[name].cpu().pin_memory() for name, _, _ in inputs.LLAMA70B_PROJ}
        hA = {k: v.cpu().pin_memory() for k, v in A_dec.items()}
        hC = {k: torch.empty(v.shape, dtype=torch.float32).pin_memory() for k, v in C_dec.items()}

        def e2e_step():
            for M in inputs.LLAMA_DECODE_M:
                for name, K, N in inputs.LLAMA70B_PROJ:
                    tl.gemm_host(hA[name, M], hW[name], hC[name, M], M, N, K, scratch, G, BR, BC)
                    tl.read_amp(M, N, K, plans[name, M].cta, tl.LAYOUT_TILE_MAJOR, G, BR, BC, 2)
        e2e_step()
        n_e2e = max(1, min(args.steps, 3))
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n_e2e):
            e2e_step()
        b.record()
        torch.cuda.synchronize()
        e_ms = a.elapsed_time(b) / n_e2e
        h2d = sum(2 * K * N + 2 * M * K for _, K, N in inputs.LLAMA70B_PROJ for M in inputs.LLAMA_DECODE_M)
        d2h = sum(4 * M * N for _, K, N in inputs.LLAMA70B_PROJ for M in inputs.LLAMA_DECODE_M) + 12 * 24
        # same byte accounting as the device-resident step: each call relayouts and multiplies once
        e_bytes = sum(relayout_bytes(N, K) + gemm_bytes(M, N, K) for _, K, N in inputs.LLAMA70B_PROJ
                      for M in inputs.LLAMA_DECODE_M)
        e2e = {"value": world * e_bytes / (e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": n_e2e,
               "note": "12 tl_gemm_host calls per step; every call copies A and the row-major weight from pinned host "
                       "memory, relayouts, multiplies and copies C back"}
        del scratch, hW
    except Exception as exc:  # report, never hide
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
               "error": f"{type(exc).__name__}: {exc}"}

    # ---- CPU oracle on a bounded sample
    try:
        import oracle as tlo
        tlo.build()
        cpu = oracle_sample(15.0)
        cpu.pop("seconds", None)
    except Exception as exc:
        cpu = {"value": None, "unit": UNIT, "cores": None, "kind": "oracle", "sample": f"failed: {exc}"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_dict(world),
        "breakdown": {"gemm_decode_GBps": gemm_gbs, "relayout_GBps": relayout_gbs,
                      "gemm_ms_per_step": g_ms / args.steps, "relayout_ms_per_step": r_ms / args.steps},
        "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": launches_per_step * args.steps, "extra": extra,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


PROFILE_CASES = {
    # name: (kind, M, K, N) -- small single-kernel cases for ncu captures (a few hundred MB on the device)
    "decode_qkv_m8": ("gemm", 8, 8192, 10240),
    "decode_o_m32": ("gemm", 32, 8192, 8192),
    "decode_down_m1": ("gemm", 1, 28672, 8192),
    "mid_gate_up_m128": ("gemm", 128, 8192, 57344),         # 128 x 256 x 64 tiles, whole tiles on 112 CTAs
    "mid_gate_up_m256": ("gemm", 256, 8192, 57344),         # 256 x 256 x 64: two token blocks per weight slab
    "prefill_o": ("gemm", 4096, 8192, 8192),
    "prefill_qkv": ("gemm", 4096, 8192, 10240),
    "relayout_o": ("relayout", 0, 8192, 8192),
    "moe_gate_up": ("moe", 0, 2048, 1536),
    "moe_down": ("moe", 0, 768, 2048),
    "kmajor_decode_qkv_m8": ("kmajor", 8, 8192, 10240),     # weights [N][K], (64, 32) memory tiles of Eq. 2
    "fp8_decode_qkv_m8": ("fp8", 8, 8192, 10240),           # E4M3, 64 x 64 memory tiles
    "fp8_prefill_o": ("fp8", 4096, 8192, 8192),             # E4M3, 64 x 64 memory tiles, CTA-pair kernel
    "hw_box_load_o": ("hw", 0, 8192, 8192),                 # every 64 x 256 box of the weight through a 2-D view
    "generic_16x8_m16": ("generic", 16, 8192, 8192),        # 16 x 8 memory tiles, permuting generic-address path (switch)
    "as_stored_16x8_m16": ("as_stored", 16, 8192, 8192),    # 16 x 8 memory tiles (16-byte rows) read as they are
    "in_place_32x4_m16": ("in_place_32x4", 16, 8192, 8192), # 32 x 4 memory tiles (8-byte rows): fetched as stored, fixed up in place
    "in_place_8x2_m16": ("in_place_8x2", 16, 8192, 8192),   # 8 x 2 memory tiles (4-byte rows)
    "relayout_layer": ("relayout_batch", 0, 0, 0),          # the four Llama weights in one launch (3.4 GB resident)
}


def run_case(args):
    """Runs one named kernel `--steps` times on cuda:0 (tile-major, default tile); prints nothing timed."""
    from paper_2607_04031_b200 import binding as tl
    kind, M, K, N = PROFILE_CASES[args.case]
    dev = "cuda:0"
    torch.cuda.set_device(0)
    if kind == "moe":
        q = inputs.QWEN_MOE
        offsets, _, _ = inputs.zipf_topk_routing(q["tokens"], q["experts"], q["topk"], q["zipf_alpha"], seed=0)
        rows = int(offsets[-1])
        Bm = inputs.bf16_normal((q["experts"], K, N), 0.02, seed=400, device=dev)
        Bt = torch.empty_like(Bm)
        tl.relayout(Bm, Bt, q["experts"] * K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
        Am = inputs.bf16_normal((rows, K), 1.0, seed=401, device=dev)
        Cm = torch.empty((rows, N), dtype=torch.float32, device=dev)
        d_off = torch.from_numpy(offsets).to(dev)
        for _ in range(args.steps):
            tl.gemm_grouped(Am, Bt, Cm, d_off, q["experts"], rows, N, K, G, BR, BC)
    elif kind == "relayout_batch":
        srcs = [inputs.bf16_normal((k, n), 0.02, seed=100 + i, device=dev) for i, (_, k, n) in enumerate(inputs.LLAMA70B_PROJ)]
        dsts = [torch.empty_like(t) for t in srcs]
        for _ in range(args.steps):
            tl.relayout_batch(srcs, dsts, [(k, n) for _, k, n in inputs.LLAMA70B_PROJ], 2, G, BR, BC, tl.TO_TILE_MAJOR)
    elif kind in ("generic", "as_stored") or kind.startswith("in_place"):
        if kind == "generic":
            tl.set_option(tl.OPT_GENERIC_RAW, 0)            # the permuting path, which these tiles no longer take by default
        br, bc = (16, 8) if not kind.startswith("in_place") else tuple(int(x) for x in kind.split("_")[2].split("x"))
        W = inputs.bf16_normal((K, N), 0.02, seed=100, device=dev)
        Wt = torch.empty_like(W)
        tl.relayout(W, Wt, K, N, 2, br * bc * 2, br, bc, tl.TO_TILE_MAJOR)
        A = inputs.bf16_normal((M, K), 1.0, seed=200, device=dev)
        C = torch.empty((M, N), dtype=torch.float32, device=dev)
        for _ in range(args.steps):
            tl.gemm(A, Wt, C, M, N, K, br * bc * 2, br, bc)
    elif kind in ("kmajor", "hw"):
        w = inputs.bf16_normal((N, K), 0.02, seed=100, device=dev)
        wt = torch.empty_like(w)
        tl.relayout(w, wt, N, K, 2, G, 32, 64, tl.TO_TILE_MAJOR)
        if kind == "kmajor":
            A = inputs.bf16_normal((M, K), 1.0, seed=200, device=dev)
            C = torch.empty((M, N), dtype=torch.float32, device=dev)
            for _ in range(args.steps):
                tl.gemm_kmajor(A, wt, C, M, N, K, G, 32, 64)
        else:
            dst = torch.empty(K * N, dtype=torch.bfloat16, device=dev)
            coords = torch.tensor([[i, j] for j in range(0, N, 256) for i in range(0, K, 64)], dtype=torch.int32, device=dev)
            desc = tl.hw_desc([K, N], [1, K], [64, 256], 2, 64, 32, K)
            for _ in range(args.steps):
                tl.hw_box_load(desc, wt, coords, dst)
    elif kind == "fp8":
        w = inputs.fp8_normal((N, K), 0.05, seed=100, device=dev).view(torch.uint8)
        wt = torch.empty_like(w)
        tl.relayout(w, wt, N, K, 1, G, 64, 64, tl.TO_TILE_MAJOR)
        A = inputs.fp8_normal((M, K), 1.0, seed=200, device=dev).view(torch.uint8)
        C = torch.empty((M, N), dtype=torch.float32, device=dev)
        for _ in range(args.steps):
            tl.gemm_fp8_kmajor(A, wt, C, M, N, K, G, 64, 64)
    else:
        W = inputs.bf16_normal((K, N), 0.02, seed=100, device=dev)
        Wt = torch.empty_like(W)
        for _ in range(args.steps if kind == "relayout" else 1):
            tl.relayout(W, Wt, K, N, 2, G, BR, BC, tl.TO_TILE_MAJOR)
        if kind == "gemm":
            A = inputs.bf16_normal((M, K), 1.0, seed=200, device=dev)
            C = torch.empty((M, N), dtype=torch.float32, device=dev)
            for _ in range(args.steps):
                if args.layout == "row":
                    tl.gemm(A, W, C, M, N, K, 0, 0, 0)
                else:
                    tl.gemm(A, Wt, C, M, N, K, G, BR, BC)
    tl.device_status()
    print(json.dumps({"case": args.case, "layout": args.layout, "launches": args.steps, "status": "ok"}), flush=True)


def run_sweep(args):
    """Config 5: N = K = 8192 bf16 weight, M in {1, 16, 128}; G x block aspect x CTA tile.
    Prints one JSON line per (G, block, CTA tile): exact read amplification (row-major vs tile-major) and
    GEMM time / throughput per M.  Weights rotate over three copies (403 MB) so every launch is L2-cold."""
    from paper_2607_04031_b200 import binding as tl
    torch.cuda.set_device(0)
    dev = "cuda:0"
    K = N = 8192
    copies = 3
    W = [inputs.bf16_normal((K, N), 0.02, seed=700 + c, device=dev) for c in range(copies)]
    Wt = [torch.empty_like(w) for w in W]
    A = {M: inputs.bf16_normal((M, K), 1.0, seed=710 + M, device=dev) for M in (1, 16, 128)}
    C = {M: torch.empty((M, N), dtype=torch.float32, device=dev) for M in (1, 16, 128)}

    def timed(M, buf_list, g, br, bc, cta, reps=4):
        evs = []
        for rep in range(reps + 1):
            for c in range(copies):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                tl.gemm(A[M], buf_list[c], C[M], M, N, K, g, br, bc, cta)
                b.record()
                if rep:
                    evs.append((a, b))
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in evs) * 1e3      # us

    # "CTA tile X x Y" of the workload list is token rows x weight columns; the K step is the kernel's own: 128 weight
    # rows per stage for the 64- and 128-column tiles (half as many barrier hand-offs per byte: 64 x 64 runs at 3.1
    # instead of 2.4 TB/s), 64 for the 256-token tile, whose token side already fills the stage
    ctas = ((64, 64, 128), (128, 128, 128), (256, 128, 64))
    for _ in range(200):                                     # clocks up before anything is timed
        tl.gemm(A[128], W[0], C[128], 128, N, K, 0, 0, 0, ctas[1])
    torch.cuda.synchronize()
    for g in (32, 256, 1024, 4096, 16384):
        for br in (1, 8, 16, 32):
            bc = g // (2 * br)
            if bc < 1:
                print(json.dumps({"G": g, "block": [br, "G/(2*%d) < 1" % br], "skipped": "block row shorter than one element"}))
                continue
            for c in range(copies):
                tl.relayout(W[c], Wt[c], K, N, 2, g, br, bc, tl.TO_TILE_MAJOR)
            # the library's rule: 1-row tiles are row-major; tile rows of at least 32 bytes are TMA boxes (128-byte
            # swizzle from 64 columns, 64-/32-byte swizzle for 32/16 columns); shorter rows are hand-addressed
            # (of those, tiles with 16-byte rows and single-column tiles of at least 8 rows are fetched as stored)
            path = ("row-major view" if br == 1 else "tma" if bc >= 64 else
                    "tma, %d-byte swizzle" % (bc * 2) if bc in (16, 32) else
                    "tma, tiles as stored" if bc == 8 and br >= 8 else
                    "tma, K-major panels" if bc == 1 and br >= 8 else
                    "tma as stored + in-place transpose" if bc in (2, 4) and br >= 8 else "generic-address")
            # the row-major times every row is compared with are taken next to it (same minute, same clocks)
            base = {(cta, M): timed(M, W, 0, 0, 0, cta) for cta in ctas for M in (1, 16, 128)}
            for cta in ctas:
                ra_t = tl.read_amp(128, N, K, cta, tl.LAYOUT_TILE_MAJOR, g, br, bc, 2)
                ra_r = tl.read_amp(128, N, K, cta, tl.LAYOUT_ROW_MAJOR, g, 0, 0, 2)
                row = {"G": g, "block": [br, bc], "cta": list(cta), "path": path,
                       "read_amp_tile_major": ra_t[0] / ra_t[1], "read_amp_row_major": ra_r[0] / ra_r[1],
                       "requests_per_load_tile_major": ra_t[2] // (ra_t[1] // (cta[2] * cta[1] * 2)),
                       "requests_per_load_row_major": ra_r[2] // (ra_r[1] // (cta[2] * cta[1] * 2))}
                try:
                    for M in (1, 16, 128):
                        us = timed(M, Wt, g, br, bc, cta)
                        row[f"M{M}_us"] = round(us, 1)
                        row[f"M{M}_GBps"] = round(gemm_bytes(M, N, K) / us / 1e3)
                        row[f"M{M}_vs_row_major_time"] = round(us / base[cta, M], 3)
                    row["generic_path"] = tl.gemm_last_plan().generic_path
                except tl.TileLensError as exc:
                    row["gemm"] = f"unsupported: {exc}"
                print(json.dumps(row), flush=True)
    tl.device_status()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--sweep", action="store_true", help="layout/granularity sweep on an 8192 x 8192 weight")
    ap.add_argument("--case", default=None, choices=sorted(PROFILE_CASES),
                    help="run one small kernel case --steps times (for ncu); no benchmark line")
    ap.add_argument("--layout", default="tile", choices=["tile", "row"])
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)      # ~0.3 s timed: long enough for clock samples inside it
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
