#!/usr/bin/env python
"""Benchmark of the fused sigmoid-attention forward + backward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl ours|reference]

A "step" is one forward plus one backward pass over one synthetic batch of the chosen
configuration (default c4: causal LM shape B=2, H=16, N=4096, D=128, bf16, QK-normed
inputs, b = -log N).  Metric: useful bf16 TFLOP/s of the step, FLOPs counted as
4 c B H N^2 D (forward) + 10 c B H N^2 D (backward), c = (N+1)/(2N) when causal.

One JSON line is printed by rank 0.  With N > 1 (torchrun), every rank runs the same
workload on its own GPU and its own batch (the (batch, head) pairs are independent, no
collective exists on the path): weak scaling, value = FLOPs of all ranks / max time.

`--impl reference` times the float64 CPU oracle on the host cores instead (a bounded
sample of the same workload); it is a deliberately slow baseline, not a target.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2409_04431_b200 import inputs, sharding  # noqa: E402

METRIC = "sigmoid-attn fwd+bwd bf16 TFLOP/s"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}
L2_FLUSH_BYTES = 256 << 20

# DRAM bytes per launch of each kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture per kernel and workload) are kept in a small data file next to the profile summaries
# they come from, so that a refreshed capture updates the bench line without touching this file.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def ncu_traffic(kernel: str, workload: str):
    """Measured DRAM bytes per launch of `kernel` ("fwd" or "bwd_main") on `workload`, or None."""
    try:
        with open(TRAFFIC_FILE) as f:
            entry = json.load(f)["kernels"][kernel][workload]
        return float(entry["dram_bytes_read"]) + float(entry["dram_bytes_write"])
    except (OSError, KeyError, ValueError, TypeError):
        return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def blas_threads_all_cores():
    """Let numpy's BLAS use every host core of this process (torchrun exports OMP_NUM_THREADS=1 to
    its ranks, which would otherwise time the oracle on one core) and return the thread count in use."""
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        threadpool_limits(limits=host_cores(), user_api="blas")
        counts = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(counts) if counts else 1
    except Exception:  # noqa: BLE001 - without threadpoolctl the environment decides
        env = os.environ.get("OMP_NUM_THREADS")
        return int(env) if env and env.isdigit() else host_cores()


# ----------------------------------------------------------------------------- oracle legs


def oracle_sample(cfg, budget_s: float = 20.0):
    """Time the float64 oracle, as it stands, on a bounded sample of `cfg`: whole heads of
    one batch element, as many as fit the time budget (at least one)."""
    import oracle  # test infrastructure; used here for the CPU baseline only

    threads = blas_threads_all_cores()
    q, k, v, d_o = inputs.make_inputs(cfg, heads=1, batch=1)
    slopes = cfg.slopes()
    sl = None if slopes is None else slopes[:1]
    rb = 1024 if cfg.N > 4096 else None
    t0 = time.perf_counter()
    oracle.sigattn_fwd(q, k, v, cfg.scale, cfg.bias, cfg.causal, sl, row_block=rb)
    oracle.sigattn_bwd(q, k, v, d_o, cfg.scale, cfg.bias, cfg.causal, sl, row_block=rb)
    one = time.perf_counter() - t0
    heads = max(1, min(cfg.B * cfg.H, int(budget_s / max(one, 1e-6))))
    total = one
    done = 1
    while done < heads:
        t0 = time.perf_counter()
        oracle.sigattn_fwd(q, k, v, cfg.scale, cfg.bias, cfg.causal, sl, row_block=rb)
        oracle.sigattn_bwd(q, k, v, d_o, cfg.scale, cfg.bias, cfg.causal, sl, row_block=rb)
        total += time.perf_counter() - t0
        done += 1
    flops_head = (cfg.flops_fwd() + cfg.flops_bwd()) / (cfg.B * cfg.H)
    return {
        "value": flops_head * done / total / 1e12,
        "unit": UNIT,
        "cores": threads,
        "kind": "oracle",
        "sample": f"{done} of {cfg.B * cfg.H} (batch, head) pairs of {cfg.name}, fwd+bwd, float64 numpy, "
                  f"{total:.1f} s wall",
    }, total / done


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, args.steps)
    warm = max(0, args.warmup)
    per_step_budget = 90.0 / (steps + warm)   # whole run: about 1.5 minutes plus one head per step at least
    vals, times = [], []
    base = None
    for s in range(warm + steps):
        base, per_head = oracle_sample(cfg, budget_s=per_step_budget)
        if s >= warm:
            vals.append(base["value"])
            times.append(per_head)
    value = float(np.mean(vals))
    base["value"] = value
    line = {
        "impl": "reference",
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warm,
        "ms_per_step": float(np.mean(times)) * 1e3 * cfg.B * cfg.H,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args.gpus),
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def algorithmic_bytes(cfg):
    """Compulsory HBM bytes of one forward and of one backward: every [B, H, N, D] tensor once
    (forward: Q, K, V in, O out; backward: Q, K, V, dO in, dQ, dK, dV out) plus the three passes
    (clear, accumulate, convert) over the fp32 dQ accumulator."""
    t = cfg.B * cfg.H * cfg.N * cfg.D
    e = 2 if cfg.dtype == "bf16" else 4
    return 4 * t * e, 7 * t * e + 3 * t * 4


def workload_config(cfg, n_gpus):
    return {
        "workload": f"{cfg.name}: B={cfg.B} H={cfg.H} N={cfg.N} D={cfg.D} {cfg.dtype} "
                    f"{'causal' if cfg.causal else 'full'}{' alibi' if cfg.alibi else ''}"
                    f"{' qk-norm' if cfg.qk_norm else ''} b=-ln(N), one fwd+bwd per step",
        "per_gpu_batch": cfg.B, "gpus": n_gpus,
        "cache": f"L2 flushed between timed steps (write of {L2_FLUSH_BYTES >> 20} MiB)",
    }


# ----------------------------------------------------------------------------- clocks


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.stop_flag = threading.Event()
        self.sm, self.reasons, self.max_sm = [], set(), None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self.stop_flag.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self):
        if not self.ok or not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_sm, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.sm)), "sm_max_mhz": self.max_sm, "reasons": sorted(self.reasons),
                "samples": len(self.sm)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        parts = [p for p in vis.split(",") if p.strip() != ""]
        try:
            return int(parts[local_index])
        except (ValueError, IndexError):
            return local_index
    return local_index


# ----------------------------------------------------------------------------- our arm


def time_side_workload(sa, torch, dev, cfg, steps, flush, peaks, bias=None, sampler_index=None):
    """Forward and backward of one further configuration, timed like the headline one: seeded host
    inputs copied to the device, >= 3 warm-up steps, L2 flushed before every timed step, CUDA events
    around each pass, clocks sampled while it runs.  Returns the per-pass figures for the bench line."""
    code = 0 if cfg.dtype == "bf16" else 1
    bias = cfg.bias if bias is None else bias
    host = inputs.make_inputs(cfg)
    q, k, v, d_o = (torch.from_numpy(inputs.f32_to_bf16_bits(x).view(np.int16)).view(torch.bfloat16).to(dev)
                    for x in host)
    del host
    o = torch.empty_like(q)
    grads = tuple(torch.empty_like(q) for _ in range(3))
    sl = cfg.slopes()
    slopes = None if sl is None else torch.from_numpy(sl).to(dev)
    ws = torch.empty(max(1, sa.sigattn_bwd_workspace_bytes(cfg.B, cfg.H, cfg.N, cfg.D, code)), dtype=torch.uint8,
                     device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    k0, k1 = ev(), ev()
    k0.record(); k1.record()
    torch.cuda.synchronize()
    for _ in range(3):
        sa.sigattn_fwd(q, k, v, cfg.scale, bias, cfg.causal, slopes, out=o)
        sa.sigattn_bwd(q, k, v, d_o, cfg.scale, bias, cfg.causal, slopes, workspace=ws, out=grads)
    sa.sigattn_check()
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    e0, e1, e2 = [ev() for _ in range(steps)], [ev() for _ in range(steps)], [ev() for _ in range(steps)]
    torch.cuda.synchronize()
    launches0 = sa.sigattn_launch_count()
    if sampler:
        sampler.start()
    kern = []
    spin = getattr(torch.cuda, "_sleep", None)   # (a private helper of torch: used when present)
    for s in range(steps):
        flush.zero_()
        # A short spin on the device (it touches no memory) lets the host enqueue the whole step before the
        # device reaches it: the smallest configuration runs 0.03 ms per pass, less than the host needs to
        # issue one, and the events would otherwise time the host.
        if spin is not None:
            spin(200_000)
        e0[s].record()
        sa.sigattn_fwd(q, k, v, cfg.scale, bias, cfg.causal, slopes, out=o)
        e1[s].record()
        timed = s % 4 == 0
        if timed:
            sa.sigattn_bwd_set_timing_events(k0, k1)
        sa.sigattn_bwd(q, k, v, d_o, cfg.scale, bias, cfg.causal, slopes, workspace=ws, out=grads)
        if timed:
            sa.sigattn_bwd_set_timing_events(None, None)
        e2[s].record()
        if timed:
            torch.cuda.synchronize()
            kern.append(k0.elapsed_time(k1))
    torch.cuda.synchronize()
    if sampler:
        sampler.stop_flag.set()
        sampler.join()
    sa.sigattn_check()
    launches = sa.sigattn_launch_count() - launches0
    t_fwd = float(np.median([e0[s].elapsed_time(e1[s]) for s in range(steps)]))
    t_bwd = float(np.median([e1[s].elapsed_time(e2[s]) for s in range(steps)]))
    t_kern = float(np.median(kern))
    peak, hbm = peaks["bf16_tflops"], peaks["hbm_gbs"]
    bytes_fwd, bytes_bwd = algorithmic_bytes(cfg)
    f_fwd, f_bwd = cfg.flops_fwd(), cfg.flops_bwd()
    out = {
        "workload": workload_config(cfg, 1)["workload"] if bias == cfg.bias else
                    workload_config(cfg, 1)["workload"].replace("b=-ln(N)", f"b={bias:g}"),
        "steps": steps, "timing": "median of per-step CUDA-event times, L2 flushed before every step, step enqueued "
                                  "behind a 0.1 ms device-side spin so that host launch time is not counted",
        "fwd": {"ms": t_fwd, "tflops": f_fwd / t_fwd / 1e9, "frac_of_peak": f_fwd / t_fwd / 1e9 / peak,
                "hbm_gbs": bytes_fwd / t_fwd / 1e6, "frac_of_hbm_peak": bytes_fwd / t_fwd / 1e6 / hbm},
        "bwd": {"ms": t_bwd, "tflops": f_bwd / t_bwd / 1e9, "frac_of_peak": f_bwd / t_bwd / 1e9 / peak,
                "hbm_gbs": bytes_bwd / t_bwd / 1e6, "frac_of_hbm_peak": bytes_bwd / t_bwd / 1e6 / hbm,
                "main_kernel_ms": t_kern, "main_kernel_tflops": f_bwd / t_kern / 1e9,
                "main_kernel_frac_of_peak": f_bwd / t_kern / 1e9 / peak},
        "gpu_launches": int(launches),
    }
    if sampler:
        out["clocks"] = sampler.summary()
    return out



def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import paper_2409_04431_b200 as sa  # raises if libsigattn.so is missing: no fallback

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    steps, warm = max(1, args.steps), max(3, args.warmup)
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    code = 0 if cfg.dtype == "bf16" else 1

    # host inputs (seeded; each rank its own batch) -> pinned host tensors -> device
    qh, kh, vh, doh = inputs.make_inputs(cfg, seed=sharding.rank_seed(cfg, rank))

    def to_torch_host(x):
        if cfg.dtype == "bf16":
            t = torch.from_numpy(inputs.f32_to_bf16_bits(x).view(np.int16)).view(torch.bfloat16)
        else:
            t = torch.from_numpy(x)
        return t.pin_memory()

    host_in = [to_torch_host(x) for x in (qh, kh, vh, doh)]
    host_out = [torch.empty_like(host_in[0]).pin_memory() for _ in range(4)]
    q, k, v, d_o = (t.to(dev, non_blocking=True) for t in host_in)
    o = torch.empty_like(q)
    grads = tuple(torch.empty_like(q) for _ in range(3))
    slopes_np = cfg.slopes()
    slopes = None if slopes_np is None else torch.from_numpy(slopes_np).to(dev)
    slopes_host = None if slopes_np is None else torch.from_numpy(slopes_np).pin_memory()
    ws = torch.empty(max(1, sa.sigattn_bwd_workspace_bytes(cfg.B, cfg.H, cfg.N, cfg.D, code)), dtype=torch.uint8,
                     device=dev)
    arena = torch.empty(sa.sigattn_step_host_arena_bytes(cfg.B, cfg.H, cfg.N, cfg.D, code), dtype=torch.uint8,
                        device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    def fwd():
        sa.sigattn_fwd(q, k, v, cfg.scale, cfg.bias, cfg.causal, slopes, out=o)

    def bwd():
        sa.sigattn_bwd(q, k, v, d_o, cfg.scale, cfg.bias, cfg.causal, slopes, workspace=ws, out=grads)

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    sampled = list(range(0, steps, 8))          # steps whose main backward kernel is timed on its own
    k_ev = {s: (ev(), ev()) for s in sampled}
    for a, b in k_ev.values():                  # create the handles before handing them to the library
        a.record(); b.record()
    torch.cuda.synchronize()

    for _ in range(warm):
        fwd(); bwd()
    sa.sigattn_check()

    # ---- timed region: K steps, device-resident inputs, L2 flushed between steps (untimed)
    sampler = ClockSampler(physical_gpu_index(local))
    e_fwd0, e_fwd1, e_bwd1 = [ev() for _ in range(steps)], [ev() for _ in range(steps)], [ev() for _ in range(steps)]
    barrier()
    launches0 = sa.sigattn_launch_count()
    sampler.start()
    wall0 = time.perf_counter()
    for s in range(steps):
        flush.zero_()
        e_fwd0[s].record()
        fwd()
        e_fwd1[s].record()
        if s in k_ev:  # the hook adds two event records around the main kernel
            sa.sigattn_bwd_set_timing_events(*k_ev[s])
            bwd()
            sa.sigattn_bwd_set_timing_events(None, None)
        else:
            bwd()
        e_bwd1[s].record()
    barrier()
    kern_ms = [a.elapsed_time(b) for a, b in k_ev.values()]
    wall = time.perf_counter() - wall0
    launches = sa.sigattn_launch_count() - launches0
    sampler.stop_flag.set()
    sampler.join()
    sa.sigattn_check()

    fwd_ms = [e_fwd0[s].elapsed_time(e_fwd1[s]) for s in range(steps)]
    bwd_ms = [e_fwd1[s].elapsed_time(e_bwd1[s]) for s in range(steps)]
    t_fwd, t_bwd = float(np.sum(fwd_ms)), float(np.sum(bwd_ms))
    t_total = t_fwd + t_bwd

    # ---- end to end: host (pinned) inputs -> device -> fwd + bwd -> host, through the C ABI
    e2e_steps = max(3, min(steps, 10))
    for _ in range(2):
        sa.sigattn_step_host(*host_in, *host_out, cfg.scale, cfg.bias, cfg.causal, slopes_host, arena=arena)
    barrier()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(e2e_steps):
        sa.sigattn_step_host(*host_in, *host_out, cfg.scale, cfg.bias, cfg.causal, slopes_host, arena=arena)
    e1.record()
    barrier()
    sa.sigattn_check()
    t_e2e = e0.elapsed_time(e1) / e2e_steps

    # max over ranks
    t_total, t_fwd, t_bwd, t_e2e, t_kern = sharding.max_over_ranks(
        [t_total, t_fwd, t_bwd, t_e2e, float(np.mean(kern_ms))], device=dev)

    if rank == 0:
        peaks, peak_src = load_peaks()
        f_fwd, f_bwd = cfg.flops_fwd(), cfg.flops_bwd()
        per_step_ms = t_total / steps
        value = sharding.whole_job_tflops(f_fwd + f_bwd, steps, world, t_total)
        fwd_tf = f_fwd * steps / (t_fwd * 1e-3) / 1e12
        bwd_tf = f_bwd * steps / (t_bwd * 1e-3) / 1e12
        kern_tf = f_bwd / (t_kern * 1e-3) / 1e12
        peak = peaks["bf16_tflops"]
        peak_sus = peaks.get("bf16_tflops_sustained", peak)   # context: cuBLAS held for seconds under the power cap
        tensor_bytes = cfg.B * cfg.H * cfg.N * cfg.D * (2 if cfg.dtype == "bf16" else 4)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": per_step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": workload_config(cfg, world),
            "fwd": {"tflops": fwd_tf, "ms": t_fwd / steps, "frac_of_peak": fwd_tf / peak,
                    "frac_of_sustained_peak": fwd_tf / peak_sus},
            "bwd": {"tflops": bwd_tf, "ms": t_bwd / steps, "frac_of_peak": bwd_tf / peak,
                    "frac_of_sustained_peak": bwd_tf / peak_sus,
                    "includes": "dQ-accumulator clear + main kernel + dQ convert"},
            "frac_of_peak": value / world / peak,
            "roofline": {
                "kernel": "sigattn_bwd_bf16_kernel (backward main kernel)",
                "bound": "tensor", "achieved": kern_tf, "peak": peak, "unit": "TFLOP/s", "frac": kern_tf / peak,
                "peak_source": f"{peak_src} bf16_tflops (burst)", "peak_sustained": peak_sus,
                "frac_of_sustained_peak": kern_tf / peak_sus, "avg_launch_ms": t_kern,
                "algorithmic_flops_per_launch": f_bwd,
                "traffic": ncu_traffic("bwd_main", cfg.name),
            },
            # the forward is one launch of one kernel, so its CUDA-event time is the kernel's
            "roofline_fwd": {
                "kernel": "sigattn_fwd_bf16_kernel (the forward is this one launch)",
                "bound": "tensor", "achieved": fwd_tf, "peak": peak, "unit": "TFLOP/s", "frac": fwd_tf / peak,
                "peak_source": f"{peak_src} bf16_tflops (burst)", "peak_sustained": peak_sus,
                "frac_of_sustained_peak": fwd_tf / peak_sus, "avg_launch_ms": t_fwd / steps,
                "algorithmic_flops_per_launch": f_fwd,
                "traffic": ncu_traffic("fwd", cfg.name),
            },
            "e2e": {"value": world * (f_fwd + f_bwd) / (t_e2e * 1e-3) / 1e12, "unit": UNIT,
                    "ms_per_step": t_e2e, "h2d_bytes_per_step": 4 * tensor_bytes, "d2h_bytes_per_step": 4 * tensor_bytes},
            "gpu_launches": int(launches),
            "clocks": sampler.summary(),
            "wall_s_timed_region": wall,
        }
        if world == 1 and not args.no_side_workloads:
            # the other bf16 configurations and the exact activation path (b = 0), same timing rules;
            # reported beside the headline, never folded into `value`
            del q, k, v, d_o, o, grads, ws, arena
            torch.cuda.empty_cache()
            side = {}
            idx = physical_gpu_index(local)
            for name in ("c2", "c3", "c5"):
                if name == cfg.name:
                    continue
                c = inputs.CONFIGS[name]
                side[name] = time_side_workload(sa, torch, dev, c, 30 if name == "c5" else 100, flush, peaks,
                                                sampler_index=idx)
                for kern in ("fwd", "bwd_main"):
                    side[name][kern.split("_")[0]]["ncu_dram_bytes_per_launch"] = ncu_traffic(kern, name)
            # every logit block on the exact path: same shape as the headline, bias 0 instead of -ln N
            side[cfg.name + "_exact_path"] = time_side_workload(sa, torch, dev, cfg, 50, flush, peaks, bias=0.0,
                                                                sampler_index=idx)
            line["workloads"] = side
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"], _ = oracle_sample(cfg, budget_s=args.cpu_budget)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_kvshard(args):
    """Strong scaling of ONE long causal sequence whose keys and values are sharded over the ranks
    (workload: the c5 shape; every rank holds all queries and its own contiguous shard of K, V and owns
    the same range of query rows).  Two arms per step, forward + backward each:
      unfused  local shard call, then one NCCL all-reduce of the fp32 summands of O and of dQ;
      fused    the kernels add into the owners' fp32 accumulators through peer mappings, owners convert.
    Sigmoid attention has no row normalisation, so the summands simply add (no log-sum-exp exchange).
    One JSON line from rank 0; times are the slowest rank's (CUDA events around each arm)."""
    import torch
    import torch.distributed as dist

    import paper_2409_04431_b200 as sa

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    cfg = inputs.CONFIGS["c5"]
    B, H, N, D = cfg.B, cfg.H, cfg.N, cfg.D
    g = torch.Generator(device=dev).manual_seed(20240904)      # the same tensors on every rank
    q, k, v, d_o = (((torch.randn(B, H, N, D, device=dev, generator=g) * cfg.std).to(torch.bfloat16)) for _ in range(4))
    owners = [sharding.kv_shard_range(N, world, r) for r in range(world)]
    mine = owners[rank]
    ks, vs = k[:, :, mine.start:mine.stop].contiguous(), v[:, :, mine.start:mine.stop].contiguous()
    q_sl = [q[:, :, r.start:r.stop].contiguous() for r in owners]
    do_sl = [d_o[:, :, r.start:r.stop].contiguous() for r in owners]
    starts = [r.start for r in owners]
    n_own = mine.stop - mine.start
    acc = torch.zeros((2, B, H, n_own, D), dtype=torch.float32, device=dev)
    peers = sharding.PeerAccumulators(acc)
    half = [B * H * (r.stop - r.start) * D * 4 for r in owners]
    o_addr = [peers.address(r, 0) for r in range(world)]
    dq_addr = [peers.address(r, half[r]) for r in range(world)]
    dk, dv = torch.empty_like(ks), torch.empty_like(vs)
    ws = torch.empty(sa.sigattn_bwd_workspace_bytes(B, H, N, D, 0), dtype=torch.uint8, device=dev)
    steps, warm = max(1, args.steps), max(3, args.warmup)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def unfused():
        o = sa.sigattn_fwd_shard(q, ks, vs, cfg.scale, cfg.bias, -mine.start, True).float()
        dq, gk, gv, _ = sa.sigattn_bwd_shard(q, ks, vs, d_o, cfg.scale, cfg.bias, -mine.start, True, workspace=ws)
        dq = dq.float()
        if world > 1:
            dist.all_reduce(o)
            dist.all_reduce(dq)
        return o.to(torch.bfloat16), dq.to(torch.bfloat16), gk, gv

    def fused():
        acc.zero_()
        barrier()                                       # every accumulator is clear before anyone adds
        sharding.kv_sharded_fwd_acc(
            lambda a, b, c, dst, pos0: sa.sigattn_fwd_shard_acc(a, b, c, dst, cfg.scale, cfg.bias, pos0, True),
            q_sl, starts, ks, vs, mine.start, o_addr)
        sharding.kv_sharded_bwd_acc(
            lambda a, b, c, d, dst, gk, gv, pos0: sa.sigattn_bwd_shard_acc_kv(a, b, c, d, dst, gk, gv, cfg.scale,
                                                                            cfg.bias, pos0, True),
            q_sl, do_sl, starts, ks, vs, mine.start, dq_addr, dk, dv)
        peers.all_added()
        return sa.sigattn_acc_to_bf16(acc[0]), sa.sigattn_acc_to_bf16(acc[1], cfg.scale), dk, dv

    times = {}
    for name, fn in (("unfused", unfused), ("fused", fused)):
        for _ in range(warm):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        sa.sigattn_check()
        times[name] = sharding.max_over_ranks([e0.elapsed_time(e1) / steps], device=dev)[0]
    peers.close()
    if rank == 0:
        flops = cfg.flops_fwd() + cfg.flops_bwd()
        line = {
            "metric": METRIC, "value": flops / (times["fused"] * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": warm, "ms_per_step": times["fused"], "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"kvshard: one causal sequence B={B} H={H} N={N} D={D} bf16, keys and values in "
                                   f"{world} contiguous shards, one fwd+bwd per step", "gpus": world,
                       "cache": "inputs of 0.5 GB per tensor (larger than L2), no flush"},
            "fused": {"ms_per_step": times["fused"], "tflops": flops / (times["fused"] * 1e-3) / 1e12,
                      "how": "kernels add into the owners' fp32 accumulators through peer mappings; host barrier "
                             "before the owners convert (inside the timed step)"},
            "unfused": {"ms_per_step": times["unfused"], "tflops": flops / (times["unfused"] * 1e-3) / 1e12,
                        "how": "local shard kernels, then NCCL all-reduce of the fp32 summands of O and dQ"},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(inputs.CONFIGS) + ["kvshard"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true",
                    help="skip the c2/c3/c5 and exact-path figures that follow the headline measurement")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    if args.workload == "kvshard":
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the kvshard workload has no CPU arm; use --workload c5"}))
            return
        run_kvshard(args)
        return
    cfg = inputs.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
