#!/usr/bin/env python
"""Benchmark of the fused AdaGC + AdamW step (Algorithm 1 of arXiv 2502.11034) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
                    [--parallel replicas|sharded]

A step is one pass of the whole path (norm -> clip decision / gamma update -> AdamW on the clipped
gradient) over every tensor of a synthetic, seeded layout; the default layout is shaped like
Llama-2 7B (291 tensors, 6.74e9 parameters, bf16 gradients, fp32 parameters and moments).  Timed
steps are steady-state AdaGC steps (t > T_start).  One JSON line is printed by rank 0:

  value        parameters/s over all GPUs, inputs resident in HBM, CUDA-event time, max over ranks
  e2e          the same metric through the host-buffer entry point (gradients copied from pinned host
               memory and per-tensor statistics copied back inside the timed region)
  roofline     the update kernel: algorithmic bytes (26 B/param with bf16 gradients, 28 with fp32)
               over its measured duration, against the measured HBM copy bandwidth
  cpu_baseline the CPU oracle timed on a bounded sample of the same layout (N=1 only)

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the step on
its own GPU: after the data-parallel gradient all-reduce the optimizer step needs no exchange, so there
is no collective on the data path ("replicas only", weak scaling).  `--impl reference` times the CPU
oracle instead of the CUDA library.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "fused AdaGC+AdamW step time, params/s, HBM GB/s (% of peak) at 7B layout"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the update kernel, per parameter, from the committed
# captures of the same kernel on smaller layouts (a multi-pass capture is not pointed at a 94 GB workload); scaled by the
# parameter count because the traffic of this streaming kernel grows in proportion.  None once a kernel has changed
# since its capture.
TRAFFIC_BYTES_PER_PARAM = {   # (gradient dtype, state dtype) -> (bytes per parameter, capture)
    ("bf16", "f32"): ((1742.350e6 + 1434.920e6) / 124439808,
                      "profiles/adagc_kernels_gpt2_small_ncu_full.md (GPT-2-small-shaped layout, scaled by N)"),
    ("bf16", "bf16"): ((1244.628e6 + 937.533e6) / 124439808,
                       "profiles/adagc_kernels_gpt2_small_ncu_full.md (GPT-2-small-shaped layout, bfloat16 state, scaled by N)"),
    ("f32", "f32"): ((3077.705e6 + 2248.135e6) / 191408576,
                     "profiles/adagc_kernels_many_small_ncu_full.md (20 000 small tensors, scaled by N)"),
}


# ------------------------------------------------------------------------------------ helpers
def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(x: float, device) -> float:
    """MAX all-reduce of one scalar (identity when not distributed)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job units/s: every rank processes `units_per_rank`, time is the max over ranks."""
    return units_per_rank * world / seconds_max


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            ident = str(device_index)
        self.cmd = ["nvidia-smi", "-i", ident, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                    "-lms", "100"]

    def start(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def bytes_per_param(wl) -> int:
    return 26 if wl.grad_dtype == "bf16" else 28


def workload_config(wl):
    return {"workload": f"{wl.name}: {wl.n_tensors} tensors, {wl.n_params} params, {wl.grad_dtype} grads, "
                        f"fp32 params/m/v ({wl.notes})",
            "n_params": wl.n_params, "n_tensors": wl.n_tensors, "grad_dtype": wl.grad_dtype,
            "hyper": {k: wl.hyper[k] for k in ("lr", "beta1", "beta2", "eps", "wd", "lambda_rel", "beta",
                                               "lambda_abs")},
            "l2": "working set far larger than L2 (no flush needed)" if wl.n_params * 14 > (1 << 30)
                  else "L2 flushed between timed steps"}


# ------------------------------------------------------------------------------------ reference arm
def oracle_sample(wl, max_params=8.2e8):
    """Bounded sample of the layout for the CPU oracle: the leading tensors up to ~max_params
    (for the Llama-2-7B-shaped layout: the first four transformer layers, embedding skipped)."""
    tensors = [t for t in wl.tensors if not t.name.startswith(("embed", "wte"))]
    picked, tot = [], 0
    for t in tensors:
        if tot + t.numel > max_params and picked:
            break
        picked.append(t)
        tot += t.numel
    return picked, tot


def time_oracle(wl, steps: int, warm: int, sample=None):
    """Times the C oracle, as it stands, on the bounded sample; returns (params/s, s/step, info)."""
    from oracle import c_oracle
    picked, tot = sample if sample is not None else oracle_sample(wl)
    offs, o = [], 0
    for t in picked:
        offs.append(o)
        o += (t.numel + 7) // 8 * 8
    nums = [t.numel for t in picked]
    rng = np.random.RandomState(7)
    theta0 = (rng.standard_normal(o) * 0.02).astype(np.float32)
    hp = wl.hyper
    ref = c_oracle.ArenaOracle(offs, nums, theta0, lr=hp["lr"], beta1=hp["beta1"], beta2=hp["beta2"],
                               eps=hp["eps"], wd=hp["wd"], lambda_rel=hp["lambda_rel"], beta=hp["beta"],
                               lambda_abs=hp["lambda_abs"], warmup=1)
    g32 = (rng.standard_normal(o) * wl.grad_scale).astype(np.float32)
    if wl.grad_dtype == "bf16":
        g = torch.from_numpy(g32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()
    else:
        g = g32
    del g32
    for _ in range(max(warm, 1)):
        ref.step(g)
    t0 = time.perf_counter()
    for _ in range(steps):
        ref.step(g)
    dt = time.perf_counter() - t0
    cpu_model = None
    try:
        with open("/proc/cpuinfo") as f:
            cpu_model = next((ln.split(":", 1)[1].strip() for ln in f if ln.startswith("model name")), None)
    except OSError:
        pass
    info = {"kind": "oracle", "cores": c_oracle.num_threads(), "cpu_model": cpu_model,
            "sample": f"{steps} step(s) of the C oracle over {len(picked)} tensors "
                      f"({picked[0].name}..{picked[-1].name}, {tot} params) of {wl.name}"}
    return tot * steps / dt, dt / steps, info


def oracle_extra_legs(wl, g_host, sample_params_per_s):
    """Further legs of the CPU baseline, each labelled with what it covers:
      all_norms      the oracle's phase 1 + 2 over ALL tensors of the layout (sums of squares streamed from the host copy
                     of the gradient arena, then the decisions), i.e. everything of a step that needs no optimizer state;
      single_thread  the whole oracle step on a smaller sample with one OpenMP thread;
      extrapolated   seconds per full step = all_norms + (update time per parameter on the sample) x N."""
    import ctypes
    from oracle import c_oracle
    out = {}
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    g_np = g_host.view(torch.int16).numpy().view(np.uint16) if g_host.dtype == torch.bfloat16 else g_host.numpy()
    gamma = np.zeros(wl.n_tensors, np.float32)
    t0 = time.perf_counter()
    ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
    c_oracle.clip_decisions(ssq, gamma, 2, wl.hyper["lambda_rel"], wl.hyper["beta"], wl.hyper["lambda_abs"], 1)
    dt = time.perf_counter() - t0
    out["all_norms"] = {"seconds": dt, "value": wl.n_params / dt, "unit": UNIT, "cores": c_oracle.num_threads(),
                        "sample": f"norm + decision phases of the C oracle over all {wl.n_tensors} tensors "
                                  f"({wl.n_params} params) of {wl.name}, one step"}
    # update cost per parameter on the sample: its whole step minus its own norm phase
    picked, tot = oracle_sample(wl)
    t0 = time.perf_counter()
    c_oracle.sumsq_tensors(g_np, np.array([t.offset for t in picked], np.int64), np.array([t.numel for t in picked], np.int64))
    norm_sample = time.perf_counter() - t0
    upd_per_param = max(tot / sample_params_per_s - norm_sample, 0.0) / tot
    full = dt + upd_per_param * wl.n_params
    out["extrapolated_full_layout"] = {"seconds_per_step": full, "value": wl.n_params / full, "unit": UNIT,
                                       "sample": "extrapolated: all_norms (measured on the full layout) + the sample's "
                                                 "update time per parameter x all parameters"}
    try:
        gomp = ctypes.CDLL("libgomp.so.1")
        n_before = c_oracle.num_threads()
        gomp.omp_set_num_threads(1)
        small, stot = oracle_sample(wl, max_params=1.2e8)
        val1, _, info1 = time_oracle(wl, 1, 1, sample=(small, stot))
        gomp.omp_set_num_threads(n_before)
        out["single_thread"] = {"value": val1, "unit": UNIT, "cores": 1, "sample": info1["sample"]}
    except OSError:
        out["single_thread"] = None
    return out


def run_reference(args, wl):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))
    val, sec, info = time_oracle(wl, steps, 1)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": 1, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(wl),
            "cpu_baseline": dict(info, value=val, unit=UNIT),
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def time_layout(binding, workloads, wl, dev, steps, warm=3, state_dtype=torch.float32, fused_small=False):
    """One layout on one GPU, the way the headline number is taken: `warm` untimed steps, then `steps` steady-state AdaGC
    steps timed with CUDA events (L2 flushed before each step when the layout is small), then the same number of steps
    with the library's per-phase events.  Returns milliseconds and fractions of the minimum-bytes roofline."""
    hp = wl.hyper
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=dev, state_dtype=state_dtype)
    theta = workloads.init_params(wl, dev)
    m = torch.zeros(wl.arena_elems, dtype=state_dtype, device=dev)
    v = torch.zeros_like(m)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)
    g = workloads.grads_for_step(wl, 1, dev)
    small = wl.n_params * 14 <= (1 << 30)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None
    args_h = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], 1)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t = 0
    per, ph = [], []
    for k in range(warm + 2 * steps):
        t += 1
        timed, phased = warm <= k < warm + steps, k >= warm + steps
        opt.set_phase_timing(phased)
        if flush is not None:
            flush.fill_(t & 0xFF)
        if timed:
            e0.record()
        opt.step(theta, g, m, v, ema, t, *args_h)
        if timed:
            e1.record()
            e1.synchronize()
            per.append(e0.elapsed_time(e1))
        if phased:
            ph.append(opt.get_phase_times())
    opt.set_phase_timing(False)
    peak, _ = measured_peak()
    sb = 2 if state_dtype == torch.bfloat16 else 4
    gb = 2 if wl.grad_dtype == "bf16" else 4
    bpp = 8 + gb + 4 * sb                       # theta read + written, g read, m and v read + written
    ms = float(np.median(per))
    norm_ms, fin_ms, upd_ms = (float(x) for x in np.median(np.array(ph), axis=0))
    out = {"n_params": wl.n_params, "n_tensors": wl.n_tensors, "grad_dtype": wl.grad_dtype,
           "state_dtype": "bf16" if sb == 2 else "f32", "min_bytes_per_param": bpp, "ms_per_step": ms,
           "norm_ms": norm_ms, "finalize_ms": fin_ms, "update_ms": upd_ms,
           "update_kernel_frac_of_measured": bpp * wl.n_params / (upd_ms * 1e-3) / 1e9 / peak,
           "norm_kernel_frac_of_measured": gb * wl.n_params / (norm_ms * 1e-3) / 1e9 / peak,
           "whole_step_frac_of_measured": bpp * wl.n_params / (ms * 1e-3) / 1e9 / peak,
           "whole_step_frac_of_nominal_8TBs": bpp * wl.n_params / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
           "l2": "flushed before every step" if small else "working set far larger than L2"}
    t_bpp, t_src = TRAFFIC_BYTES_PER_PARAM.get((wl.grad_dtype, out["state_dtype"]), (None, None))
    out["update_kernel_traffic"] = t_bpp * wl.n_params if t_bpp else None        # ncu DRAM bytes per launch, scaled by N
    out["update_kernel_traffic_source"] = t_src
    if fused_small and opt.n_chunks <= 4096:
        # launch-latency-bound layouts: wall clock over back-to-back steps like a training loop, the default step (two
        # launches) against the one-kernel step (ADAGC_FUSED_SMALL)
        fused = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=dev, flags=binding.FUSED_SMALL,
                              state_dtype=state_dtype)
        ema_f = torch.zeros_like(ema)
        for name, o, e_ in (("default_step_us_back_to_back", opt, ema), ("fused_small_step_us_back_to_back", fused, ema_f)):
            tt = 100
            for _ in range(20):
                tt += 1
                o.step(theta, g, m, v, e_, tt, *args_h)
            torch.cuda.synchronize(dev)
            w0 = time.perf_counter()
            for _ in range(200):
                tt += 1
                o.step(theta, g, m, v, e_, tt, *args_h)
            torch.cuda.synchronize(dev)
            out[name] = (time.perf_counter() - w0) / 200 * 1e6
        fused.close()
    assert opt.get_stats()["status"] == 0
    opt.close()
    return out


# ------------------------------------------------------------------------------------ our arm
def run_ours(args, wl):
    from paper_2502_11034_b200 import binding, workloads
    import torch.distributed as dist

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    hp = wl.hyper
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=dev)
    theta = workloads.init_params(wl, dev)
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)
    g = workloads.grads_for_step(wl, 1, dev)
    small = wl.n_params * 14 <= (1 << 30)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None
    args_h = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"])
    T_START = 1        # step 1 is a warm-up (global-norm) step that seeds gamma; all later steps are AdaGC steps
    t = 0

    def one_step():
        nonlocal t
        t += 1
        if flush is not None:
            flush.fill_(t & 0xFF)
        opt.step(theta, g, m, v, ema, t, *args_h, T_START)

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    n_warm = max(args.warmup, 3)
    for _ in range(n_warm):
        one_step()
    sync_all()

    # ---- timed region: K steady-state steps, device-resident inputs
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    launches0 = opt.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    if small:
        per = []
        for _ in range(args.steps):
            flush.fill_(1)
            e0.record()
            t += 1
            opt.step(theta, g, m, v, ema, t, *args_h, T_START)
            e1.record()
            e1.synchronize()
            per.append(e0.elapsed_time(e1) * 1e-3)
        seconds = sum(per)
    else:
        e0.record()
        for _ in range(args.steps):
            one_step()
        e1.record()
        e1.synchronize()
        seconds = e0.elapsed_time(e1) * 1e-3
    sync_all()
    launches = opt.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    seconds_max = max_over_ranks(seconds, dev)
    value = job_throughput(wl.n_params * args.steps, world, seconds_max)

    # ---- per-kernel durations (CUDA events recorded by the library on the launching stream)
    opt.set_phase_timing(True)
    ph = []
    for _ in range(args.steps):
        one_step()
        ph.append(opt.get_phase_times())
    opt.set_phase_timing(False)
    norm_ms, fin_ms, upd_ms = (float(x) for x in np.array(ph).mean(axis=0))
    peak, peak_kind = measured_peak()
    bpp = bytes_per_param(wl)
    step_s = seconds_max / args.steps
    achieved = bpp * wl.n_params / (upd_ms * 1e-3) / 1e9
    norm_gbs = (bpp - 24) * wl.n_params / (norm_ms * 1e-3) / 1e9
    kernel = "adagc_update_tma_kernel" if opt.update_path == binding.UPDATE_PATH_BULK else "adagc_update_kernel"
    traffic_bpp, traffic_src = TRAFFIC_BYTES_PER_PARAM.get((wl.grad_dtype, "f32"), (None, None))
    if kernel != "adagc_update_tma_kernel":
        traffic_bpp, traffic_src = None, None
    whole_gbs = bpp * wl.n_params / step_s / 1e9
    roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                "traffic": traffic_bpp * wl.n_params if traffic_bpp else None,
                "traffic_source": traffic_src,
                "algorithmic_bytes_per_launch": bpp * wl.n_params, "launch_ms": upd_ms,
                # the whole step against the minimum bytes the method must move (g read once): the step reads g twice
                # (norm pass, update pass), so its ceiling is 26/28 (28/32 with fp32 gradients) of the bandwidth reached
                "whole_step": {"achieved": whole_gbs, "frac_of_measured": whole_gbs / peak,
                               "frac_of_nominal_8TBs": whole_gbs / NOMINAL_HBM_GBS,
                               "target_frac_of_nominal": 0.80, "target_met": bool(whole_gbs / NOMINAL_HBM_GBS >= 0.80),
                               "min_bytes_per_param": bpp, "bytes_moved_per_param": bpp + (2 if wl.grad_dtype == "bf16" else 4)},
                "whole_step_frac": whole_gbs / peak,
                "whole_step_frac_of_nominal_8TBs": whole_gbs / NOMINAL_HBM_GBS,
                "norm_kernel": {"launch_ms": norm_ms, "achieved": norm_gbs, "frac": norm_gbs / peak},
                "finalize_ms": fin_ms}

    # ---- a warm-up (global-norm) step and the clip-only entry, reported separately
    extra = {}
    e0.record()
    opt.step(theta, g, m, v, ema, 1, *args_h, 10 ** 9)      # step <= T_start: global-norm branch (re-seeds gamma)
    e1.record(); e1.synchronize()
    extra["warmup_branch_step_ms"] = e0.elapsed_time(e1)
    g_out = torch.empty_like(g)
    for name, dst in (("clip_only_out_of_place_ms", g_out), ("clip_only_in_place_ms", g)):
        opt.clip(g, dst, ema, 2, hp["lambda_rel"], hp["beta"], T_START)
        torch.cuda.synchronize(dev)
        e0.record()
        opt.clip(g, dst, ema, 3, hp["lambda_rel"], hp["beta"], T_START)
        e1.record(); e1.synchronize()
        extra[name] = e0.elapsed_time(e1)
    del g_out
    # the clip fused with Lion (one state stream: 18 B/param with bf16 gradients, 20 with fp32)
    opt.set_phase_timing(True)
    for k in range(3):
        opt.step_lion(theta, g, m, ema, 4 + k, 1e-4, 0.9, 0.99, hp["wd"], hp["lambda_rel"], hp["beta"], T_START)
    lion_ms = opt.get_phase_times()
    opt.set_phase_timing(False)
    lion_bpp = bpp - 8
    extra["lion_step_ms"] = sum(lion_ms)
    extra["lion_update_kernel"] = {"launch_ms": lion_ms[2], "achieved": lion_bpp * wl.n_params / (lion_ms[2] * 1e-3) / 1e9,
                                   "frac": lion_bpp * wl.n_params / (lion_ms[2] * 1e-3) / 1e9 / peak}

    # the step that also emits the bf16 working copy of the parameters (28 B/param with bf16 gradients)
    if all(t_.offset % 8 == 0 for t_ in wl.tensors):
        lowp = torch.empty(wl.arena_elems, dtype=torch.bfloat16, device=dev)
        opt.set_phase_timing(True)
        for k in range(3):
            opt.step_emit_bf16(theta, lowp, g, m, v, ema, 7 + k, *args_h, T_START)
        emit_ms = opt.get_phase_times()
        opt.set_phase_timing(False)
        extra["emit_bf16_step_ms"] = sum(emit_ms)
        extra["emit_bf16_update_kernel"] = {"launch_ms": emit_ms[2],
                                            "achieved": (bpp + 2) * wl.n_params / (emit_ms[2] * 1e-3) / 1e9,
                                            "frac": (bpp + 2) * wl.n_params / (emit_ms[2] * 1e-3) / 1e9 / peak}
        del lowp

    # ---- end to end through the host-buffer entry point
    e2e_steps = max(1, min(args.steps, 5))
    g_host = torch.empty(wl.arena_elems, dtype=wl.torch_grad_dtype).pin_memory()
    g_host.copy_(g)
    T = wl.n_tensors
    hn, hh = torch.empty(T, dtype=torch.float32).pin_memory(), torch.empty(T, dtype=torch.float32).pin_memory()
    hf = torch.empty(T, dtype=torch.uint8).pin_memory()
    t += 1
    opt.step_host(theta, g, m, v, ema, g_host, t, *args_h, T_START, hn, hh, hf)
    sync_all()
    w0 = time.perf_counter()
    for _ in range(e2e_steps):
        t += 1
        opt.step_host(theta, g, m, v, ema, g_host, t, *args_h, T_START, hn, hh, hf)   # synchronises itself
    e2e_sec = max_over_ranks(time.perf_counter() - w0, dev)
    e2e = {"value": job_throughput(wl.n_params * e2e_steps, world, e2e_sec), "unit": UNIT,
           "h2d_bytes_per_step": g_host.numel() * g_host.element_size(), "d2h_bytes_per_step": T * 9,
           "steps": e2e_steps, "ms_per_step": e2e_sec / e2e_steps * 1e3,
           "note": "wall clock around adagc_step_host (it synchronises the stream); gradients from pinned host memory"}
    st = opt.get_stats()
    assert st["status"] == 0 and np.isfinite(st["norm"]).all()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        val, sec, info = time_oracle(wl, 5, 1)
        cpu_baseline = dict(info, value=val, unit=UNIT)
        cpu_baseline.update(oracle_extra_legs(wl, g_host, val))
    del g_host

    # ---- the same step with the moments stored as bfloat16 (18 B/param instead of 26), and the other layouts
    if world == 1 and not args.no_extras:
        del theta, m, v, g, ema
        opt.close()
        torch.cuda.empty_cache()
        k = max(3, min(args.steps, 10))
        if all(t_.offset % 8 == 0 for t_ in wl.tensors):
            r = time_layout(binding, workloads, wl, dev, k, 3, torch.bfloat16)
            extra["bf16_state"] = r
            extra["bf16_state_update_kernel"] = {"launch_ms": r["update_ms"], "bytes_per_param": r["min_bytes_per_param"],
                                                 "achieved": r["min_bytes_per_param"] * wl.n_params / (r["update_ms"] * 1e-3) / 1e9,
                                                 "frac": r["update_kernel_frac_of_measured"]}
        if args.workload is None:
            per_config = {}
            for name in ("llama32_1b", "gpt2_small", "many_small", "tiny"):
                torch.cuda.empty_cache()
                per_config[name] = time_layout(binding, workloads, workloads.build(name), dev, 20, 5,
                                               fused_small=(name == "tiny"))
            for name in ("moe_8x1b", "moe_ernie"):      # expert-parallel-shaped layouts: 747 and 3828 tensors
                torch.cuda.empty_cache()
                wl_x = workloads.build(name)
                need = wl_x.arena_elems * 14 + (6 << 30)       # theta, m, v, bf16 g, and room for the generator's scratch
                free, _ = torch.cuda.mem_get_info()
                if free < need:
                    per_config[name] = {"skipped": f"needs {need >> 30} GiB of free device memory, {free >> 30} GiB free"}
                else:
                    per_config[name] = time_layout(binding, workloads, wl_x, dev, 5, 3)
            extra["per_config"] = per_config

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": n_warm, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(wl), parallelism=f"replicas x{world} (no collective)"),
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
                "cpu_baseline": cpu_baseline, "extra": extra}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_sharded(args, wl):
    """--parallel sharded: the layout's arenas cut into N flat shards, one per rank; each step is
    adagc_shard_sumsq -> all-reduce of n_tensors float64 (NCCL) -> adagc_step_presummed.  Total work is fixed as N
    grows (strong scaling); with N = 1 it measures what the split of the step costs."""
    from paper_2502_11034_b200 import binding, sharded, workloads
    import torch.distributed as dist

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    hp = wl.hyper
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    opt = sharded.ShardedAdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], rank, world, device=dev)
    n_local = max(opt.local_elems, 8)
    gen = torch.Generator(device=dev)
    gen.manual_seed(workloads.BASE_SEED + rank)
    theta = torch.empty(n_local, device=dev).normal_(0.0, 0.02, generator=gen)
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    g = torch.empty(n_local, device=dev).normal_(0.0, wl.grad_scale, generator=gen).to(wl.torch_grad_dtype)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)
    args_h = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if n_local * 14 <= (1 << 30) else None
    t = 0

    def one_step():
        nonlocal t
        t += 1
        if flush is not None:
            flush.fill_(t & 0xFF)
        opt.step(theta, g, m, v, ema, t, *args_h, 1)

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    n_warm = max(args.warmup, 3)
    for _ in range(n_warm):
        one_step()
    sync_all()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    launches0 = opt.opt.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for _ in range(args.steps):
        one_step()
    e1.record()
    e1.synchronize()
    seconds = e0.elapsed_time(e1) * 1e-3
    sync_all()
    clocks = sampler.stop() if sampler else None
    seconds_max = max_over_ranks(seconds, dev)
    st = opt.opt.get_stats()
    assert st["status"] == 0 and st["steps_done"] == t
    if rank == 0:
        peak, peak_kind = measured_peak()
        bpp = bytes_per_param(wl)
        step_s = seconds_max / args.steps
        line = {"metric": METRIC, "value": wl.n_params * args.steps / seconds_max, "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": n_warm, "ms_per_step": step_s * 1e3, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": dict(workload_config(wl), parallelism=f"flat shards x{world}, one all-reduce of "
                                                                f"{wl.n_tensors} float64 per step"),
                "clocks": clocks, "gpu_launches": int(opt.opt.launch_count() - launches0),
                "roofline": {"bound": "hbm", "kernel": "whole sharded step", "unit": "GB/s", "peak": peak,
                             "peak_source": f"of {peak_kind}",
                             "achieved": bpp * wl.n_params / world / step_s / 1e9,
                             "frac": bpp * wl.n_params / world / step_s / 1e9 / peak, "traffic": None}}
        print(json.dumps(line), flush=True)
    opt.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def pick_workload(args):
    from paper_2502_11034_b200 import workloads
    if args.workload:
        return workloads.build(args.workload)
    wl = workloads.build("llama2_7b")
    if args.impl == "ours" and torch.cuda.is_available():
        free, _ = torch.cuda.mem_get_info(int(os.environ.get("LOCAL_RANK", "0")))
        if free < wl.arena_elems * 16 + (6 << 30):
            wl = workloads.build("llama32_1b")      # largest configuration that fits; named in config.workload
    return wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=None, help="tiny | gpt2_small | llama2_7b | many_small | llama32_1b | moe_8x1b | moe_ernie")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the bfloat16-state and other-layout measurements")
    ap.add_argument("--parallel", choices=["replicas", "sharded"], default="replicas",
                    help="N > 1: independent replicas (default; the data-parallel case) or flat shards of one model")
    args = ap.parse_args()
    wl = pick_workload(args)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.parallel == "sharded":
        run_sharded(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
