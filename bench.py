#!/usr/bin/env python
"""Benchmark of the CLEAR attention forward pass (one call = one attention layer of one denoising step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` is effective TFLOP/s, 4 * sum(M) * head_dim * H * B / time (the paper's
4 * sum(M) * c), with q, k, v resident in HBM; `e2e` is the same metric through the host-tensor C-ABI
entry point with the host<->device copies inside the timed region.  With N > 1 (torchrun) every rank runs
an independent replica of the workload on its own GPU: the path has no exchange step.
`qk_prep` times, outside `value`, the one-pass Q/K preparation kernel (normalisation + rotary embedding) on the
same shape against the HBM copy rate; `bwd` times the tensor-core backward pass of the operator.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2412_16112_b200 import workloads

METRIC = "effective TFLOP/s (4*sum(M)*c) of the CLEAR attention forward"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU while the timed region runs (read-only queries):
    through NVML every 20 ms where the Python binding is there, else through nvidia-smi (slower per sample)."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    PERIOD_S = 0.02

    def __init__(self, index: int):
        self.index = index
        self.sm, self.mx, self.power = [], [], []
        self.reasons = set()
        self.source = "nvidia-smi"
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [x.strip() for x in visible.split(",") if x.strip()]
                if index < len(ids) and ids[index].isdigit():
                    phys = int(ids[index])
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self._nvml = pynvml
            self.source = "nvml"
        except Exception:
            self._nvml = None

    def _sample_nvml(self):
        n = self._nvml
        self.sm.append(float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM)))
        self.mx.append(float(n.nvmlDeviceGetMaxClockInfo(self._handle, n.NVML_CLOCK_SM)))
        try:
            self.power.append(n.nvmlDeviceGetPowerUsage(self._handle) / 1000.0)
        except Exception:
            pass
        try:
            bits = n.nvmlDeviceGetCurrentClocksEventReasons(self._handle)
        except Exception:
            bits = n.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle)
        for name, const in (("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                            ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                            ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                            ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap")):
            if bits & getattr(n, const, 0):
                self.reasons.add(name)

    def _sample_smi(self):
        out = subprocess.run(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                              "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
        parts = [x.strip() for x in out.strip().split(",")]
        if len(parts) < 7:
            return
        self.sm.append(float(parts[0]))
        self.mx.append(float(parts[1]))
        try:
            self.power.append(float(parts[2]))
        except ValueError:
            pass
        for name, val in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], parts[3:7]):
            if val.lower().startswith("active"):
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                if self._nvml is not None:
                    self._sample_nvml()
                else:
                    self._sample_smi()
            except Exception:
                pass
            self._stop.wait(self.PERIOD_S)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": max(self.mx) if self.mx else None,
                "power_w_max": max(self.power) if self.power else None, "reasons": sorted(self.reasons),
                "samples": len(self.sm), "source": self.source}


def sample_rows_for_cpu(w, n_text_rows, n_img_rows, seed=0):
    rng = np.random.default_rng(seed)
    n = w.grid_h * w.grid_w
    rows = [(0, 0, int(i)) for i in rng.integers(0, max(w.n_text, 1), n_text_rows) if w.n_text > 0]
    rows += [(0, 0, w.n_text + int(p)) for p in rng.integers(0, n, n_img_rows)]
    return np.array(rows, dtype=np.int64)


_COUNTS_CACHE = {}


def allowed_counts(w):
    """Per-query number of allowed keys, from the oracle's own mask (cached per workload)."""
    from oracle import clear_oracle as oracle
    key = (w.grid_h, w.grid_w, w.n_text, w.radius)
    if key not in _COUNTS_CACHE:
        _COUNTS_CACHE[key] = oracle.mask_counts(w.grid_h, w.grid_w, w.n_text, w.radius)[1]
    return _COUNTS_CACHE[key]


def time_oracle_sample(w, q, k, v, target_s=15.0):
    """Oracle throughput on a bounded sample of query rows of head 0, in the metric's unit:
    4 * (allowed pairs of the sampled rows) * head_dim / seconds."""
    from oracle import clear_oracle as oracle
    counts = allowed_counts(w)
    pilot = sample_rows_for_cpu(w, 2, 64)
    t0 = time.perf_counter()
    oracle.attn_rows(q, k, v, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale, pilot)
    t_pilot = time.perf_counter() - t0
    scale_up = max(1.0, target_s / max(t_pilot, 1e-3))
    n_text_rows = max(2, int(2 * scale_up))
    n_img_rows = max(64, int(64 * scale_up))
    # the pilot includes one-off costs, so it underestimates the rate: grow the sample until it runs long enough
    for attempt in range(3):
        rows = sample_rows_for_cpu(w, n_text_rows, n_img_rows, seed=1)
        t0 = time.perf_counter()
        oracle.attn_rows(q, k, v, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale, rows)
        dt = time.perf_counter() - t0
        if dt >= 0.6 * target_s:
            break
        grow = min(8.0, target_s / max(dt, 1e-3))
        n_text_rows, n_img_rows = int(n_text_rows * grow), int(n_img_rows * grow)
    pairs = int(counts[rows[:, 2]].sum())
    tflops = 4.0 * pairs * w.head_dim / dt / 1e12
    return {"value": tflops, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{len(rows)} query rows of head 0 ({n_text_rows} text, {n_img_rows} image), "
                      f"{pairs} allowed pairs, {dt:.2f} s"}, dt, pairs


def time_oracle_full(w, q, k, v):
    """The oracle on the whole workload (every head, every row): for the workloads it finishes in seconds."""
    from oracle import clear_oracle as oracle
    pairs = int(allowed_counts(w).sum()) * w.B * w.H
    t0 = time.perf_counter()
    oracle.attn(q, k, v, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale)
    dt = time.perf_counter() - t0
    return {"value": 4.0 * pairs * w.head_dim / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"the whole workload ({pairs} allowed pairs), {dt:.2f} s"}


FULL_ORACLE_WORKLOADS = ("c0_tiny_f32", "c1_1024px_r8", "c2_2048px_r16")


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    if args.steps is None:
        args.steps = 5
    q, k, v = workloads.make_inputs(w, heads=1)
    per_step_target = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    times, pairs_all = [], []
    info = None
    for s in range(args.warmup + args.steps):
        info, dt, pairs = time_oracle_sample(w, q, k, v, target_s=per_step_target)
        if s >= args.warmup:
            times.append(dt)
            pairs_all.append(pairs)
    value = 4.0 * sum(pairs_all) * w.head_dim / sum(times) / 1e12
    info["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w), "cpu_baseline": info,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the replicas of a multi-GPU run are as fast as their slowest member."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(world: int, flops_per_replica: float, ms_per_step: float) -> float:
    """Whole-job TFLOP/s of `world` independent replicas that all take `ms_per_step` (the slowest rank's)."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


def workload_config(w):
    return {"workload": w.name, "B": w.B, "H": w.H, "head_dim": w.head_dim, "grid_h": w.grid_h, "grid_w": w.grid_w,
            "n_text": w.n_text, "radius": w.radius, "l2": "inputs larger than L2 (no flush)" if
            4 * w.B * w.H * w.n_tokens * w.head_dim * 2 > 126e6 * 2 else "L2 flushed between steps"}


def run_ours(args, w):
    from paper_2412_16112_b200 import binding as clear

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    peaks, peaks_kind = load_peaks()
    q, k, v = workloads.make_inputs(w)
    dtype_code = clear.BF16 if w.dtype == "bf16" else clear.F32
    plan = clear.Plan(w.B, w.H, w.grid_h, w.grid_w, w.n_text, w.head_dim, w.radius, dtype=dtype_code)
    info = plan.info()
    flops = info.flops
    qd, kd, vd = (t.to(dev) for t in (q, k, v))
    out = torch.empty_like(qd)
    stream = torch.cuda.current_stream()
    small = 4 * qd.numel() * qd.element_size() <= 2 * 126e6
    flush = torch.empty(int(256e6), dtype=torch.uint8, device=dev) if small else None
    launches_per_call = 1 + (1 if (info.kernel != clear.KERNEL_SIMT and info.n_text_splits > 1) else 0)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    plan.forward(qd, kd, vd, out, w.scale)
    w0.record(stream)
    for _ in range(args.warmup):
        plan.forward(qd, kd, vd, out, w.scale)
    w1.record(stream)
    plan.check()
    if args.steps is None:
        # no --steps given: as many as make the timed region last 0.6 s (same count on every rank)
        warm_ms = max_over_ranks(w0.elapsed_time(w1) / args.warmup, dist, dev)
        args.steps = int(min(2000, max(20, math.ceil(600.0 / max(warm_ms, 1e-3)))))

    # ---- device-resident timing -----------------------------------------------------------------
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    with ClockSampler(local_rank) as clocks:
        t_wall0 = time.perf_counter()
        for s in range(args.steps):
            if flush is not None:
                flush.fill_(s & 0xFF)
            ev[s][0].record(stream)
            plan.forward(qd, kd, vd, out, w.scale)
            ev[s][1].record(stream)
        barrier()
        t_wall = time.perf_counter() - t_wall0
    plan.check()
    ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = max_over_ranks(float(sum(ms)), dist, dev)
    ms_per_step = total_ms / args.steps
    value = replica_throughput(world, flops, ms_per_step)
    clock_info = clocks.summary()

    # ---- end to end: host tensors in pinned memory, copies inside the timed region ----------------
    e2e = None
    if not args.no_e2e:
        qh, kh, vh = (t.pin_memory() for t in (q, k, v))
        oh = torch.empty_like(q).pin_memory()
        n_e2e = max(1, min(args.steps, 5))
        plan.forward_host(qh, kh, vh, oh, w.scale)  # allocates the staging buffers
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(n_e2e):
            plan.forward_host(qh, kh, vh, oh, w.scale)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / n_e2e, dist, dev)
        nbytes = q.numel() * q.element_size()
        e2e = {"value": replica_throughput(world, flops, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": 3 * nbytes, "d2h_bytes_per_step": nbytes, "steps": n_e2e}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel ------------------------------------------------------------
    per_gpu_tflops = flops / (ms_per_step * 1e-3) / 1e12
    peak = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
    # DRAM bytes of one launch from the committed ncu capture (profiles/): "workload bytes" per line
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")
    if os.path.exists(tpath) and info.kernel == clear.KERNEL_TCGEN05_WS:
        try:
            with open(tpath) as f:
                for line in f:
                    parts = line.split()
                    if len(parts) == 2 and parts[0] == w.name:
                        traffic = float(parts[1])
        except Exception:
            traffic = None
    if info.kernel != clear.KERNEL_SIMT:
        roofline = {"bound": "tensor", "achieved": per_gpu_tflops, "peak": peak, "unit": "TFLOP/s",
                    "frac": per_gpu_tflops / peak, "traffic": traffic,
                    "traffic_source": "stored ncu capture of this kernel (profiles/dram_traffic_per_launch.txt)"
                    if traffic is not None else None, "peak_kind": f"{peaks_kind} bf16 burst",
                    "frac_of_sustained": per_gpu_tflops / float(peaks.get("bf16_tflops_sustained", peak)),
                    "executed_tflops": per_gpu_tflops * info.executed_pairs / info.sum_mask,
                    "geometric_efficiency": info.sum_mask / info.executed_pairs,
                    "kernel": ("clear_ws_kernel" if info.kernel == clear.KERNEL_TCGEN05_WS else "clear_tc_kernel") +
                              " (+ combine kernel inside the same events)"}
    else:
        # fp32 CUDA-core kernel: 128 FMA lanes x 2 flops per SM per clock
        alu_peak = 148 * 128 * 2 * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
        roofline = {"bound": "alu", "achieved": per_gpu_tflops, "peak": alu_peak, "unit": "TFLOP/s",
                    "frac": per_gpu_tflops / alu_peak, "traffic": traffic, "peak_kind": "148 SMs x 128 fp32 FMA lanes",
                    "kernel": "clear_simt_kernel"}

    # ---- the Q/K preparation that precedes the attention call in the model (outside `value`) -------------
    qk_prep = None
    if not args.no_prep and w.head_dim in (64, 128):
        axes = (16, 56, 56) if w.head_dim == 128 else (8, 28, 28)
        k_out = torch.empty_like(kd)
        n_prep = 20
        for _ in range(3):
            clear.clear_qk_norm_rope(qd, kd, out, k_out, w.grid_h, w.grid_w, w.n_text, axes, ntk_factor=10.0)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        p0.record(stream)
        for _ in range(n_prep):
            clear.clear_qk_norm_rope(qd, kd, out, k_out, w.grid_h, w.grid_w, w.n_text, axes, ntk_factor=10.0)
        p1.record(stream)
        torch.cuda.synchronize()
        prep_ms = p0.elapsed_time(p1) / n_prep
        prep_bytes = 4 * qd.numel() * qd.element_size()   # Q and K read once and written once
        hbm_peak = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
        qk_prep = {"kernel": "clear_qk_prep_kernel", "ms": prep_ms, "bound": "hbm", "achieved": prep_bytes / prep_ms / 1e6,
                   "peak": hbm_peak, "unit": "GB/s", "frac": prep_bytes / prep_ms / 1e6 / hbm_peak,
                   "peak_kind": f"{peaks_kind} copy", "bytes_per_launch": prep_bytes, "launches": n_prep,
                   "note": "tensors fit in L2: no HBM figure" if small else "tensors larger than L2"}
        del k_out

    # ---- the backward pass of the same operator on the tensor cores (outside `value`) ---------------------
    bwd = None
    if not args.no_bwd and w.dtype == "bf16" and w.head_dim in (64, 128):
        grads = [torch.empty_like(qd) for _ in range(3)]
        n_bwd = 3
        for _ in range(2):
            clear.clear_attn_bwd_bf16_tc(qd, kd, vd, vd, *grads, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale)
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        b0.record(stream)
        for _ in range(n_bwd):
            clear.clear_attn_bwd_bf16_tc(qd, kd, vd, vd, *grads, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale)
        b1.record(stream)
        torch.cuda.synchronize()
        clear.clear_cache_check()
        bwd_ms = b0.elapsed_time(b1) / n_bwd
        bwd_flops = 2.5 * flops   # five matrix products per allowed pair against the forward's two
        bwd = {"kernel": "clear_bwd_tc_kernel (query role + key role)", "ms": bwd_ms, "flops_per_call": bwd_flops,
               "value": bwd_flops / (bwd_ms * 1e-3) / 1e12, "unit": "effective TFLOP/s (10*sum(M)*c)",
               "frac": bwd_flops / (bwd_ms * 1e-3) / 1e12 / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])),
               "launches": 2 * n_bwd, "note": "upstream gradient = v (any bf16 data of the right shape)"}
        del grads

    cpu_baseline = None
    if not args.no_cpu:
        if w.name in FULL_ORACLE_WORKLOADS:
            cpu_baseline = time_oracle_full(w, q, k, v)
        else:
            cpu_baseline, _, _ = time_oracle_sample(w, q[:, :1].contiguous(), k[:, :1].contiguous(),
                                                    v[:, :1].contiguous())
            cpu_baseline["sample"] += "; rate of the sample, the whole workload would take " \
                                      f"{flops / (cpu_baseline['value'] * 1e12):.0f} s at it (extrapolated)"

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(w), "clocks": clock_info, "e2e": e2e,
            "gpu_launches": launches_per_call * args.steps, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "ms_min": float(min(ms)), "ms_median": float(np.median(ms)), "wall_s_timed_region": t_wall,
            "ms_x_sm_mhz": ms_per_step * clock_info["sm_mhz"] if clock_info.get("sm_mhz") else None,
            "flops_per_call": flops, "sum_mask_per_head": info.sum_mask, "parallelism": "replicas",
            "qk_prep": qk_prep, "bwd": bwd}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_bands(args, w):
    """`--parallelism bands`: ONE workload cut into row bands over the ranks (Sec. 3.4): halo exchange, the band's
    image queries, the text queries' records, all-gather and merge, all inside the timed region.  Strong scaling;
    `value` = the whole workload's flops over the slowest rank's time.  Local inputs are drawn on the device."""
    from paper_2412_16112_b200 import band_parallel as bp
    from paper_2412_16112_b200 import binding as clear

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    if w.dtype != "bf16":
        raise RuntimeError("row bands exist for the bf16 workloads")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks, peaks_kind = load_peaks()
    att = bp.BandAttention(w.B, w.H, w.grid_h, w.grid_w, w.n_text, w.head_dim, w.radius, rank, world,
                           text_mode="average" if args.text_mode == "average" else "exact")
    lay = att.lay
    gen = torch.Generator(device=dev).manual_seed(w.seed + 100 * rank)
    shape = (w.B, w.H, lay.n_local_tokens, w.head_dim)

    def draw(norm):
        x = torch.randn(shape, generator=gen, device=dev, dtype=torch.float32)
        if norm:
            x = x / torch.sqrt(x.pow(2).mean(dim=-1, keepdim=True) + 1e-6)
        return x.to(torch.bfloat16)
    qd, kd, vd = draw(True), draw(True), draw(False)
    out = torch.empty_like(qd)
    stream = torch.cuda.current_stream()
    whole = clear.Plan(w.B, w.H, w.grid_h, w.grid_w, w.n_text, w.head_dim, w.radius, host_only=True).info()
    flops = whole.flops

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    att.forward(qd, kd, vd, out, w.scale)
    w0.record(stream)
    for _ in range(args.warmup):
        att.forward(qd, kd, vd, out, w.scale)
    w1.record(stream)
    att.check()
    if args.steps is None:
        warm_ms = max_over_ranks(w0.elapsed_time(w1) / args.warmup, dist, dev)
        args.steps = int(min(2000, max(20, math.ceil(600.0 / max(warm_ms, 1e-3)))))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    with ClockSampler(local_rank) as clocks:
        for s in range(args.steps):
            ev[s][0].record(stream)
            att.forward(qd, kd, vd, out, w.scale)
            ev[s][1].record(stream)
        barrier()
    att.check()
    ms = [a.elapsed_time(b) for a, b in ev]
    ms_per_step = max_over_ranks(float(sum(ms)), dist, dev) / args.steps
    if rank == 0:
        value = flops / (ms_per_step * 1e-3) / 1e12
        peak = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        halo_bytes = 2 * (lay.halo_lo + lay.halo_hi) * w.grid_w * w.head_dim * 2 * w.B * w.H
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic (drawn on the device, per rank)",
                "config": dict(workload_config(w), parallelism=f"row bands x{world}", text_rows=args.text_mode,
                               l2="local tensors larger than L2" if 4 * qd.numel() * 2 > 2 * 126e6 else "local tensors fit in L2"),
                "clocks": clocks.summary(), "e2e": None, "gpu_launches": 4 * args.steps,
                "roofline": {"bound": "tensor", "achieved": value / world, "peak": peak, "unit": "TFLOP/s",
                             "frac": value / world / peak, "traffic": None, "peak_kind": f"{peaks_kind} bf16 burst",
                             "kernel": "clear_ws_kernel (band image plan + band text plan) + export and merge kernels"},
                "cpu_baseline": None, "flops_per_call": flops, "parallelism": "row bands",
                "halo_bytes_received_rank0": halo_bytes,
                "record_bytes_gathered": world * w.B * w.H * w.n_text * (w.head_dim + 2) * 4}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default: as many as make the timed region last 0.6 s, at least 20)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c4_8k_r16", choices=sorted(workloads.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-prep", action="store_true", help="skip the timing of the Q/K preparation kernel")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-bwd", action="store_true", help="skip the timing of the tensor-core backward pass")
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "bands"],
                    help="replicas (default): every rank runs the whole workload; bands: one workload cut into row "
                         "bands over the ranks (Sec. 3.4), strong scaling")
    ap.add_argument("--text-mode", default="exact", choices=["exact", "average"],
                    help="bands: exact merge of the text rows, or the patch-wise average of Eq. 7")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = workloads.WORKLOADS[args.workload]
    if args.impl == "reference":
        return run_reference(args, w)
    if args.parallelism == "bands":
        return run_bands(args, w)
    return run_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
