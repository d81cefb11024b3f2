"""Drives the CUDA library and the CPU oracle over the same seeded inputs and compares them.

The gradients and the initial parameters are drawn once (on the device the CUDA path runs on)
and the same bits are copied to the host for the oracle; no expected value ever comes from the
CUDA path.  Tolerances (stated by the target of this work, repeated in each test):
  clip flags, clip counts, step counter: bit-exact;
  norms, gamma, h: 1e-5 relative;  float64 sums of squares: 1e-11 relative;
  fp32 theta, m, v: per tensor ||delta||_2 <= 1e-5 ||ref||_2 and per element
  |delta| <= 1e-5 * max(|ref|, rms(ref));  bf16 clipped gradients: 1 bf16 ulp.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch

from oracle import c_oracle
from paper_2502_11034_b200 import binding, workloads

RTOL = 1e-5


def to_numpy_grads(g: torch.Tensor) -> np.ndarray:
    g = g.detach().cpu().contiguous()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()


def hyper_of(wl: workloads.Workload, **over) -> Dict[str, float]:
    hp = dict(wl.hyper)
    hp["warmup"] = wl.warmup
    hp.update(over)
    return hp


@dataclass
class ParityReport:
    steps: int = 0
    decisions: int = 0
    clipped: int = 0
    min_margin: float = math.inf
    max_norm_rel: float = 0.0
    max_gamma_rel: float = 0.0
    max_sumsq_rel: float = 0.0
    max_tensor_rel: Dict[str, float] = field(default_factory=dict)
    gamma_bit_mismatch: int = 0

    def line(self) -> str:
        return (f"steps={self.steps} decisions={self.decisions} clipped={self.clipped} "
                f"min_margin={self.min_margin:.3e} norm_rel={self.max_norm_rel:.2e} "
                f"gamma_rel={self.max_gamma_rel:.2e} gamma_bit_mismatch={self.gamma_bit_mismatch} "
                f"sumsq_rel={self.max_sumsq_rel:.2e} state_rel={self.max_tensor_rel}")


def _rel(a: np.ndarray, b: np.ndarray) -> float:
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = np.abs(a - b) / np.abs(b)
    r[(a == b)] = 0.0
    r[np.isnan(a) & np.isnan(b)] = 0.0
    return float(np.max(r)) if r.size else 0.0


def check_decisions(st, sumsq_gpu, gamma_gpu, r, rep: ParityReport, step: int):
    """Per-step comparison of what the finalize phase produced."""
    flag_ref = np.asarray(r["flag"], bool)
    if not np.array_equal(st["flag"], flag_ref):
        bad = np.nonzero(st["flag"] != flag_ref)[0]
        raise AssertionError(f"step {step}: clip decisions differ at tensors {bad[:10]} "
                             f"(margins {np.asarray(r['margin'])[bad[:10]]})")
    rep.decisions += len(flag_ref)
    rep.clipped += int(flag_ref.sum())
    rep.min_margin = min(rep.min_margin, float(np.min(r["margin"])))
    rep.max_norm_rel = max(rep.max_norm_rel, _rel(st["norm"], r["norm"]))
    rep.max_gamma_rel = max(rep.max_gamma_rel, _rel(gamma_gpu, r["gamma"]))
    rep.gamma_bit_mismatch += int((np.asarray(gamma_gpu, np.float32).view(np.uint32) !=
                                   np.asarray(r["gamma"], np.float32).view(np.uint32)).sum())
    rep.max_sumsq_rel = max(rep.max_sumsq_rel, _rel(sumsq_gpu, np.asarray(r["norm"], np.float64) ** 2))
    assert _rel(st["norm"], r["norm"]) <= RTOL, f"step {step}: norms differ"
    assert _rel(gamma_gpu, r["gamma"]) <= RTOL, f"step {step}: gamma differs"
    assert _rel(st["h"], r["h"]) <= RTOL, f"step {step}: clip factors differ"
    assert _rel(sumsq_gpu, np.asarray(r["norm"], np.float64) ** 2) <= 1e-11, f"step {step}: float64 sums of squares differ"


def check_state(name: str, got: np.ndarray, ref: np.ndarray, rep: ParityReport, what: str = ""):
    """fp32 state of one tensor: relative L2 error and per-element error."""
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    nref = float(np.linalg.norm(ref))
    d = float(np.linalg.norm(got - ref))
    rel = d / nref if nref > 0 else d
    rep.max_tensor_rel[name] = max(rep.max_tensor_rel.get(name, 0.0), rel)
    assert rel <= RTOL, f"{name} of {what}: ||delta||/||ref|| = {rel:.3e}"
    rms = nref / math.sqrt(max(ref.size, 1))
    bound = RTOL * np.maximum(np.abs(ref), rms)
    worst = np.abs(got - ref) - bound
    assert (worst <= 0).all(), f"{name} of {what}: element error {np.abs(got - ref).max():.3e} above bound"


def run_full(wl: workloads.Workload, n_steps: int, device="cuda", hyper_over: Optional[dict] = None,
             lr_schedule=None, canary: bool = True, flags: int = 0, gamma0: Optional[float] = None,
             emit_bf16: bool = False, ema_cap: float = 0.0, capturable: str = "") -> ParityReport:
    """Every element of every tensor, fused AdaGC+AdamW step, GPU vs C oracle."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = [t.offset for t in wl.tensors]
    nums = [t.numel for t in wl.tensors]
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], device=device, flags=flags)
    if ema_cap > 0:
        opt.set_ema_cap(ema_cap)
    theta = workloads.init_params(wl, device)
    theta0 = theta.cpu().numpy().copy()
    pad_mask = None
    if canary and wl.arena_elems != wl.n_params:
        pad = np.ones(wl.arena_elems, bool)
        for o, n in zip(offs, nums):
            pad[o:o + n] = False
        pad_mask = torch.from_numpy(pad).to(device)
        theta[pad_mask] = 777.0
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    if pad_mask is not None:
        m[pad_mask] = 777.0
        v[pad_mask] = 777.0
    keep = bool(flags & binding.EMA_KEEP_INITIAL)
    # without the keep-initial variant the incoming gamma must be ignored at t = 1: poison it
    ema = torch.full((wl.n_tensors,), float("nan") if not keep else float(gamma0), dtype=torch.float32, device=device)
    ref = c_oracle.ArenaOracle(offs, nums, theta0, lr=hp["lr"], beta1=hp["beta1"], beta2=hp["beta2"],
                               eps=hp["eps"], wd=hp["wd"], lambda_rel=hp["lambda_rel"], beta=hp["beta"],
                               lambda_abs=hp["lambda_abs"], warmup=hp["warmup"], keep_initial=keep,
                               global_adaptive=bool(flags & binding.CLIP_GLOBAL_ADAPTIVE),
                               gamma0=None if not keep else np.full(wl.n_tensors, gamma0, np.float32),
                               ema_cap=ema_cap)
    rep = ParityReport()
    lowp = torch.full((wl.arena_elems,), 7.0, dtype=torch.bfloat16, device=device) if emit_bf16 else None
    # capturable = "eager": adagc_step_capturable called every step; "graph": captured ONCE into a CUDA graph before
    # the first step and replayed for every step (gradients and eta_t are refreshed in place between replays)
    graph = g_static = lr_dev = None
    if capturable:
        lr_dev = torch.zeros(1, dtype=torch.float32, device=device)
        g_static = torch.zeros(wl.arena_elems, dtype=wl.torch_grad_dtype, device=device)
        cap_args = (theta, g_static, m, v, ema, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"],
                    hp["beta"], hp["warmup"], lr_dev)
        if capturable == "graph":
            graph = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph):
                opt.step_capturable(*cap_args)
            assert opt.get_stats()["steps_done"] == 0, "capturing must not execute a step"
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        lr = hp["lr"] if lr_schedule is None else lr_schedule(t)
        if capturable:
            g_static.copy_(g)
            lr_dev.fill_(lr)
            if graph is not None:
                graph.replay()
            else:
                opt.step_capturable(*cap_args)
        elif emit_bf16:
            opt.step_emit_bf16(theta, lowp, g, m, v, ema, t, lr, hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                               hp["lambda_rel"], hp["beta"], hp["warmup"])
        else:
            opt.step(theta, g, m, v, ema, t, lr, hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                     hp["lambda_rel"], hp["beta"], hp["warmup"])
        r = ref.step(to_numpy_grads(g), lr=lr)
        st = opt.get_stats()
        check_decisions(st, opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        rep.steps = t
    st = opt.get_stats()
    assert st["steps_done"] == n_steps
    assert np.array_equal(st["clip_count"], ref.clip_count)
    assert st["status"] == 0
    th, mm, vv = theta.cpu().numpy(), m.cpu().numpy(), v.cpu().numpy()
    for t_, o, n in zip(wl.tensors, offs, nums):
        check_state("theta", th[o:o + n], ref.theta[o:o + n], rep, t_.name)
        check_state("m", mm[o:o + n], ref.m[o:o + n], rep, t_.name)
        check_state("v", vv[o:o + n], ref.v[o:o + n], rep, t_.name)
    if emit_bf16:
        # the emitted working copy is the bf16 rounding of the fp32 master: exactly so for the GPU's own theta,
        # and within one bf16 ulp of the rounding of the oracle's theta
        got = to_numpy_grads(lowp)
        for t_, o, n in zip(wl.tensors, offs, nums):
            own = to_numpy_grads(theta[o:o + n].to(torch.bfloat16))
            assert np.array_equal(got[o:o + n], own), f"bf16 copy of {t_.name} is not the rounding of theta"
            # vs the oracle: one bf16 ulp for the rounding, plus the tolerance of the fp32 theta underneath
            a = bf16_bits_to_f64(got[o:o + n])
            b = ref.theta[o:o + n].astype(np.float64)
            rms = float(np.linalg.norm(b)) / math.sqrt(max(b.size, 1))
            bound = np.abs(b) * 2.0 ** -7 + RTOL * np.maximum(np.abs(b), rms)
            assert (np.abs(a - b) <= bound).all(), f"bf16 parameters of {t_.name} differ from the oracle's theta"
        if pad_mask is not None:
            assert bool((lowp[pad_mask].float() == 7.0).all()), "bf16 copy: padding between tensors was written"
    if pad_mask is not None:
        for a in (theta, m, v):
            assert bool((a[pad_mask] == 777.0).all()), "guard bands between tensors were overwritten"
    opt.close()
    return rep


def sample_indices(numel: int, k: int, rng: np.random.RandomState, chunk: int = 16384) -> np.ndarray:
    """Element indices of one tensor to check: both ends, around chunk boundaries, and random ones."""
    idx = [np.arange(min(numel, 32)), np.arange(max(0, numel - 32), numel)]
    for b in (chunk, 2 * chunk, (numel // chunk) * chunk):
        if 0 < b < numel:
            idx.append(np.arange(max(0, b - 9), min(numel, b + 9)))
    if numel > 64:
        idx.append(rng.randint(0, numel, size=k))
    return np.unique(np.concatenate(idx)).astype(np.int64)


def run_sampled(wl: workloads.Workload, n_steps: int, device="cuda", k: int = 2048,
                mode: str = "adamw", in_place: bool = True, hyper_over: Optional[dict] = None) -> ParityReport:
    """Full-size layouts: all norms / decisions / gamma against the oracle (it streams the whole
    gradient), theta/m/v (or the clipped gradient) on sampled elements the oracle computes one by one.
    Legal because, given h_i, the update of an element depends on that element only (Algorithm 1)."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device)
    rng = np.random.RandomState(99)
    samp = [sample_indices(int(n), k, rng) + int(o) for o, n in zip(offs, nums)]   # arena indices per tensor
    sizes = np.array([len(s) for s in samp], np.int64)
    soff = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.int64)
    flat = torch.from_numpy(np.concatenate(samp)).to(device)
    rep = ParityReport()
    gamma = np.zeros(wl.n_tensors, np.float32)
    clip_count = np.zeros(wl.n_tensors, np.uint64)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=device)
    if mode == "adamw":
        theta = workloads.init_params(wl, device)
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        s_theta = theta[flat].cpu().numpy().copy()
        s_m, s_v = np.zeros_like(s_theta), np.zeros_like(s_theta)
    g_out = None
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        g_np = to_numpy_grads(g)                         # the same bits, for the oracle
        s_g = np.ascontiguousarray(g_np[flat.cpu().numpy()])
        if mode == "adamw":
            opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                     hp["lambda_rel"], hp["beta"], hp["warmup"])
        else:
            g_out = g if in_place else torch.empty_like(g)
            opt.clip(g, g_out, ema, t, hp["lambda_rel"], hp["beta"], hp["warmup"])
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        clip_count += r["flag"].astype(np.uint64)
        st = opt.get_stats()
        check_decisions(st, opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        for i in range(wl.n_tensors):
            sl = slice(int(soff[i]), int(soff[i] + sizes[i]))
            if mode == "adamw":
                c_oracle.adamw_update(s_theta[sl], s_g[sl], s_m[sl], s_v[sl], float(r["h"][i]), t,
                                      hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"])
        if mode != "adamw":
            got = to_numpy_grads(g_out[flat])
            want = np.empty_like(s_g)
            for i in range(wl.n_tensors):
                sl = slice(int(soff[i]), int(soff[i] + sizes[i]))
                c_oracle.scale(s_g[sl], float(r["h"][i]), out=want[sl])
            check_clipped_grads(got, want, f"step {t}")
        rep.steps = t
        del g
    st = opt.get_stats()
    assert st["steps_done"] == n_steps and np.array_equal(st["clip_count"], clip_count) and st["status"] == 0
    if mode == "adamw":
        g_theta, g_m, g_v = (a[flat].cpu().numpy() for a in (theta, m, v))
        for i, t_ in enumerate(wl.tensors):
            sl = slice(int(soff[i]), int(soff[i] + sizes[i]))
            check_state("theta", g_theta[sl], s_theta[sl], rep, t_.name)
            check_state("m", g_m[sl], s_m[sl], rep, t_.name)
            check_state("v", g_v[sl], s_v[sl], rep, t_.name)
    opt.close()
    return rep


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def check_clipped_grads(got: np.ndarray, want: np.ndarray, what: str):
    """Clipped gradients in the gradient dtype: fp32 within 1e-5 relative, bf16 within one bf16 ulp."""
    if got.dtype == np.uint16:
        a, b = bf16_bits_to_f64(got), bf16_bits_to_f64(want)
        ulp = np.maximum(np.abs(b), 2.0 ** -126) * 2.0 ** -7     # spacing is at most 2^-7 relative
        assert (np.abs(a - b) <= ulp).all(), f"{what}: bf16 clipped gradient off by more than one ulp"
    else:
        a, b = got.astype(np.float64), want.astype(np.float64)
        assert (np.abs(a - b) <= RTOL * np.abs(b) + 1e-45).all(), f"{what}: clipped gradient differs"


LION_TIE_TOL = 1e-5      # sign(c) decided with a relative margin below this may legitimately differ


def run_full_lion(wl: workloads.Workload, n_steps: int, device="cuda", flags: int = 0, lr: float = 1e-4,
                  beta1: float = 0.9, beta2: float = 0.99, hyper_over: Optional[dict] = None) -> ParityReport:
    """Every element, clip fused with Lion (adagc_step_lion) vs the C oracle.
    m never depends on a sign decision and is compared on every element.  theta is compared with the
    usual tolerance on every element whose sign(c) was never a near-tie (relative margin >= 1e-5, the
    path's tolerance); an element with k near-ties may differ by up to 2 lr k on top of it."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device, flags=flags)
    theta = workloads.init_params(wl, device)
    m = torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=device)
    r_theta = theta.cpu().numpy().copy()
    r_m = np.zeros_like(r_theta)
    ties = np.zeros(r_theta.shape, np.uint8)
    gamma = np.zeros(wl.n_tensors, np.float32)
    clip_count = np.zeros(wl.n_tensors, np.uint64)
    rep = ParityReport()
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        opt.step_lion(theta, g, m, ema, t, lr, beta1, beta2, hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
        g_np = to_numpy_grads(g)
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        clip_count += r["flag"].astype(np.uint64)
        for i, (o, n) in enumerate(zip(offs, nums)):
            c_oracle.lion_update(r_theta[o:o + n], g_np[o:o + n], r_m[o:o + n], float(r["h"][i]), lr, beta1, beta2,
                                 hp["wd"], near_tie=ties[o:o + n], tie_tol=LION_TIE_TOL)
        st = opt.get_stats()
        check_decisions(st, opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        rep.steps = t
    st = opt.get_stats()
    assert st["steps_done"] == n_steps and np.array_equal(st["clip_count"], clip_count) and st["status"] == 0
    th, mm = theta.cpu().numpy(), m.cpu().numpy()
    n_ties = n_flipped = 0
    for t_, o, n in zip(wl.tensors, offs, nums):
        sure = ties[o:o + n] == 0
        check_state("m", mm[o:o + n], r_m[o:o + n], rep, t_.name)
        check_state("theta", th[o:o + n][sure], r_theta[o:o + n][sure], rep, t_.name)
        if not sure.all():
            d = np.abs(th[o:o + n][~sure].astype(np.float64) - r_theta[o:o + n][~sure])
            k = ties[o:o + n][~sure].astype(np.float64)
            ref = np.abs(r_theta[o:o + n][~sure].astype(np.float64))
            assert (d <= 2.0 * lr * k * 1.001 + RTOL * np.maximum(ref, 1e-3)).all(), f"theta of {t_.name}: near-tie element off"
            n_ties += int((~sure).sum())
            n_flipped += int((d > lr).sum())
    rep.max_tensor_rel["lion_near_tie_elements"] = n_ties
    rep.max_tensor_rel["lion_flipped_elements"] = n_flipped
    assert n_flipped <= n_ties                    # (elements outside the near-tie set met the strict tolerance above)
    assert n_ties <= 1e-3 * wl.n_params + 50      # near-ties are rare: this is not a loophole for real errors
    opt.close()
    return rep


def run_full_clip(wl: workloads.Workload, n_steps: int, in_place: bool, device="cuda",
                  hyper_over: Optional[dict] = None, flags: int = 0) -> ParityReport:
    """Clip-only entry, every element: clipped gradients in the gradient dtype vs the C oracle."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device, flags=flags)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=device)
    gamma = np.zeros(wl.n_tensors, np.float32)
    rep = ParityReport()
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        g_np = to_numpy_grads(g).copy()
        out = g if in_place else torch.full_like(g, 7.0)
        opt.clip(g, out, ema, t, hp["lambda_rel"], hp["beta"], hp["warmup"])
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        check_decisions(opt.get_stats(), opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        got = to_numpy_grads(out)
        for i, (o, n) in enumerate(zip(offs, nums)):
            want = c_oracle.scale(np.ascontiguousarray(g_np[o:o + n]), float(r["h"][i]))
            check_clipped_grads(got[o:o + n], want, f"step {t}, tensor {wl.tensors[i].name}")
            if float(r["h"][i]) == 1.0:
                assert np.array_equal(got[o:o + n], g_np[o:o + n])      # unclipped tensors pass through bit for bit
        if not in_place and wl.arena_elems != wl.n_params:
            pad = np.ones(wl.arena_elems, bool)
            for o, n in zip(offs, nums):
                pad[o:o + n] = False
            assert (out.float().cpu().numpy()[pad] == 7.0).all(), "padding between tensors was written"
        rep.steps = t
    opt.close()
    return rep


def run_full_sgdm(wl: workloads.Workload, n_steps: int, device="cuda", flags: int = 0, lr: float = 1e-2,
                  momentum: float = 0.9, hyper_over: Optional[dict] = None) -> ParityReport:
    """Every element, clip fused with SGD with momentum (adagc_step_sgdm) vs the C oracle."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device, flags=flags)
    theta = workloads.init_params(wl, device)
    m = torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=device)
    r_theta = theta.cpu().numpy().copy()
    r_m = np.zeros_like(r_theta)
    gamma = np.zeros(wl.n_tensors, np.float32)
    rep = ParityReport()
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        opt.step_sgdm(theta, g, m, ema, t, lr, momentum, hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
        g_np = to_numpy_grads(g)
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        for i, (o, n) in enumerate(zip(offs, nums)):
            c_oracle.sgdm_update(r_theta[o:o + n], g_np[o:o + n], r_m[o:o + n], float(r["h"][i]), lr, momentum, hp["wd"])
        check_decisions(opt.get_stats(), opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        rep.steps = t
    th, mm = theta.cpu().numpy(), m.cpu().numpy()
    for t_, o, n in zip(wl.tensors, offs, nums):
        check_state("theta", th[o:o + n], r_theta[o:o + n], rep, t_.name)
        check_state("m", mm[o:o + n], r_m[o:o + n], rep, t_.name)
    assert opt.get_stats()["status"] == 0
    opt.close()
    return rep


def run_full_sharded(wl: workloads.Workload, n_steps: int, world: int, device="cuda", mode: str = "adamw",
                     hyper_over: Optional[dict] = None, flags: int = 0) -> ParityReport:
    """The sharded step (adagc_shard_sumsq -> sum over ranks -> adagc_step_presummed / adagc_clip_presummed)
    with `world` ranks emulated one after the other on one GPU, every element against the UNSHARDED C oracle.
    Each rank has its own context over its slices (adagc_shard_plan), its own exchange buffer and its own
    replica of gamma; the ranks' partial sums are added in rank order, which is what an all-reduce computes."""
    from paper_2502_11034_b200 import sharded
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = [t.offset for t in wl.tensors]
    nums = [t.numel for t in wl.tensors]
    ranks = [sharded.ShardedAdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], r, world, device=device,
                                  flags=flags) for r in range(world)]
    assert ranks[0].elem_begin == 0 and max(rk.elem_end for rk in ranks) == max(o + n for o, n in zip(offs, nums))
    theta = workloads.init_params(wl, device)
    theta0 = theta.cpu().numpy().copy()
    pad = np.ones(wl.arena_elems, bool)
    for o, n in zip(offs, nums):
        pad[o:o + n] = False
    pad_mask = torch.from_numpy(pad).to(device)
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    for a in (theta, m, v):
        a[pad_mask] = 777.0
    emas = [torch.full((wl.n_tensors,), float("nan"), dtype=torch.float32, device=device) for _ in ranks]
    ref = c_oracle.ArenaOracle(offs, nums, theta0, lr=hp["lr"], beta1=hp["beta1"], beta2=hp["beta2"],
                               eps=hp["eps"], wd=hp["wd"], lambda_rel=hp["lambda_rel"], beta=hp["beta"],
                               lambda_abs=hp["lambda_abs"], warmup=hp["warmup"],
                               global_adaptive=bool(flags & binding.CLIP_GLOBAL_ADAPTIVE))
    gamma_ref = np.zeros(wl.n_tensors, np.float32)
    rep = ParityReport()
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        g_np = to_numpy_grads(g).copy()
        out = g if mode == "clip_in_place" else (torch.full_like(g, 7.0) if mode == "clip" else None)
        parts = [rk.local_sumsq(g[rk.elem_begin:rk.elem_end]).clone() for rk in ranks]
        total = parts[0].clone()
        for p in parts[1:]:
            total += p                                       # stands in for the all-reduce over the ranks
        for rk, ema in zip(ranks, emas):
            b, e = rk.elem_begin, rk.elem_end
            rk.sumsq.copy_(total)
            if mode == "adamw":
                rk.opt.step_presummed(theta[b:e], g[b:e], m[b:e], v[b:e], ema, rk.sumsq, t, hp["lr"], hp["beta1"],
                                      hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
            else:
                rk.opt.clip_presummed(g[b:e], out[b:e], ema, rk.sumsq, t, hp["lambda_rel"], hp["beta"], hp["warmup"])
        if mode == "adamw":
            r = ref.step(g_np)
        else:
            ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
            r = c_oracle.clip_decisions(ssq, gamma_ref, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        stats = [rk.opt.get_stats() for rk in ranks]
        check_decisions(stats[0], total.cpu().numpy(), emas[0].cpu().numpy(), r, rep, t)
        for st, ema in zip(stats[1:], emas[1:]):             # every rank took the same decisions, bit for bit
            assert np.array_equal(st["flag"], stats[0]["flag"]) and np.array_equal(st["h"], stats[0]["h"])
            assert torch.equal(ema, emas[0]) and np.array_equal(st["clip_count"], stats[0]["clip_count"])
            assert st["steps_done"] == t and st["status"] == 0
        if mode != "adamw":
            got = to_numpy_grads(out)
            for i, (o, n) in enumerate(zip(offs, nums)):
                want = c_oracle.scale(np.ascontiguousarray(g_np[o:o + n]), float(r["h"][i]))
                check_clipped_grads(got[o:o + n], want, f"step {t}, tensor {wl.tensors[i].name}")
            if mode == "clip":
                assert bool((out[pad_mask].float() == 7.0).all()), "padding between tensors was written"
        rep.steps = t
    if mode == "adamw":
        th, mm, vv = theta.cpu().numpy(), m.cpu().numpy(), v.cpu().numpy()
        for t_, o, n in zip(wl.tensors, offs, nums):
            check_state("theta", th[o:o + n], ref.theta[o:o + n], rep, t_.name)
            check_state("m", mm[o:o + n], ref.m[o:o + n], rep, t_.name)
            check_state("v", vv[o:o + n], ref.v[o:o + n], rep, t_.name)
        assert np.array_equal(stats[0]["clip_count"], ref.clip_count)
        for a in (theta, m, v):
            assert bool((a[pad_mask] == 777.0).all()), "guard bands between tensors were overwritten"
    for rk in ranks:
        rk.close()
    return rep


# ------------------------------------------------------------------------------------------------------------------
# Optimizer state stored as bfloat16 (adagc_desc.state_dtype = ADAGC_BF16)
# ------------------------------------------------------------------------------------------------------------------
def _bf16_view(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _assert_same_bf16(name: str, got_bits: np.ndarray, ref_bits: np.ndarray, what: str):
    bad = np.nonzero(got_bits != ref_bits)[0]
    assert bad.size == 0, (f"{name} of {what}: {bad.size} of {got_bits.size} stored bfloat16 values differ from the oracle's, "
                           f"first at element {bad[:3]}: {bf16_bits_to_f64(got_bits[bad[:3]])} vs {bf16_bits_to_f64(ref_bits[bad[:3]])}")


def run_bf16_state(wl: workloads.Workload, n_steps: int, optimizer: str = "adamw", teacher_forced: bool = False,
                   device="cuda", flags: int = 0, hyper_over: Optional[dict] = None, lion_lr: float = 1e-4,
                   sgd_lr: float = 1e-2, stochastic_seed: Optional[int] = None) -> ParityReport:
    """Every element with m (and v) stored as bfloat16, GPU vs the C oracle's bfloat16-state functions.

    Which bfloat16 neighbour a moment is stored as is a discrete decision, taken on both sides in the precision the
    library states for it (single precision, a fixed operation order: the oracle's fp32_decision mode, itself pinned
    to exact rational arithmetic and to the float64 definition).  So the stored m and v must be BIT-IDENTICAL to the
    oracle's on every element at every step; theta meets the fp32 tolerance (it is computed from the unrounded moments).
      free-running    both sides carry their own state for n_steps (m and v do not depend on theta, so they stay
                      bit-identical; momentum SGD's m does depend on theta and is only compared in the other mode);
      teacher_forced  before every step the GPU's theta, m, v are overwritten with the oracle's stored state (inputs
                      flow oracle -> GPU only) and every step is compared from identical stored state.
    Lion's sign(c) near-ties may move theta by 2 lr per occurrence, as in run_full_lion.
    stochastic_seed: the moments are rounded stochastically (adagc_set_state_rounding) with this seed; the random
    numbers are a function of (seed, step, arena position) that both sides compute from the generator's published
    definition, so the stored moments stay bit-identical.
    """
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device, flags=flags,
                        state_dtype=torch.bfloat16)
    if stochastic_seed is not None:
        opt.set_state_rounding(True, stochastic_seed)
    sto = dict(stochastic_seed=stochastic_seed)
    n_state = 2 if optimizer == "adamw" else 1
    assert optimizer != "sgdm" or teacher_forced, "momentum SGD's m depends on theta: compare it from identical state"
    theta = workloads.init_params(wl, device)
    r_theta = theta.cpu().numpy().copy()
    pad = np.ones(wl.arena_elems, bool)
    for o, n in zip(offs, nums):
        pad[o:o + n] = False
    pad_mask = torch.from_numpy(pad).to(device)
    GUARD = 768.0                                            # a bfloat16 value
    theta[pad_mask] = GUARD
    m = torch.zeros(wl.arena_elems, dtype=torch.bfloat16, device=device)
    v = torch.zeros_like(m)
    m[pad_mask] = GUARD
    v[pad_mask] = GUARD
    r_m = np.zeros(wl.arena_elems, np.uint16)
    r_v = np.zeros(wl.arena_elems, np.uint16)
    sign_ties = np.zeros(wl.arena_elems, np.uint8)           # Lion only
    ema = torch.full((wl.n_tensors,), float("nan"), dtype=torch.float32, device=device)
    gamma = np.zeros(wl.n_tensors, np.float32)
    clip_count = np.zeros(wl.n_tensors, np.uint64)
    rep = ParityReport()
    lr = {"adamw": hp["lr"], "lion": lion_lr, "sgdm": sgd_lr}[optimizer]

    def gpu_step(g, t):
        if optimizer == "adamw":
            opt.step(theta, g, m, v, ema, t, lr, hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"],
                     hp["beta"], hp["warmup"])
        elif optimizer == "lion":
            opt.step_lion(theta, g, m, ema, t, lr, 0.9, 0.99, hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
        else:
            opt.step_sgdm(theta, g, m, ema, t, lr, 0.9, hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])

    def oracle_update(o, n, g_np, h, t, ties):
        sl = slice(o, o + n)
        if optimizer == "adamw":
            c_oracle.adamw_update_bf16state(r_theta[sl], g_np[sl], r_m[sl], r_v[sl], h, t, lr, hp["beta1"], hp["beta2"],
                                            hp["eps"], hp["wd"], fp32_decision=True, index0=o, **sto)
        elif optimizer == "lion":
            c_oracle.lion_update(r_theta[sl], g_np[sl], r_m[sl], h, lr, 0.9, 0.99, hp["wd"], near_tie=ties[sl],
                                 tie_tol=LION_TIE_TOL, fp32_decision=True, step=t, index0=o, **sto)
        else:
            c_oracle.sgdm_update(r_theta[sl], g_np[sl], r_m[sl], h, lr, 0.9, hp["wd"], fp32_decision=True, step=t,
                                 index0=o, **sto)

    def compare(t, ties):
        th, mb, vb = theta.cpu().numpy(), _bf16_view(m), _bf16_view(v)
        for t_, o, n in zip(wl.tensors, offs, nums):
            sl = slice(int(o), int(o + n))
            what = f"{t_.name}, step {t}"
            _assert_same_bf16("m", mb[sl], r_m[sl], what)
            if n_state == 2:
                _assert_same_bf16("v", vb[sl], r_v[sl], what)
            if optimizer == "lion":
                sure = ties[sl] == 0
                check_state("theta", th[sl][sure], r_theta[sl][sure], rep, what)
                d = np.abs(th[sl][~sure].astype(np.float64) - r_theta[sl][~sure])
                k = ties[sl][~sure].astype(np.float64)
                assert (d <= 2.0 * lr * k * 1.001 + RTOL * np.maximum(np.abs(r_theta[sl][~sure]), 1e-3)).all(), \
                    f"theta of {what}: sign near-tie element off"
            else:
                check_state("theta", th[sl], r_theta[sl], rep, what)

    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        g_np = to_numpy_grads(g)
        if teacher_forced and t > 1:                         # the oracle's stored state is this step's input on both sides
            keep = theta[pad_mask].clone()
            theta.copy_(torch.from_numpy(r_theta).to(device))
            theta[pad_mask] = keep
            for dst, src in ((m, r_m), (v, r_v)):
                bits = torch.from_numpy(src.view(np.int16)).to(device).view(torch.bfloat16)
                dst.copy_(torch.where(pad_mask, dst, bits))
        gpu_step(g, t)
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        clip_count += r["flag"].astype(np.uint64)
        step_ties = np.zeros(wl.arena_elems, np.uint8) if teacher_forced else sign_ties
        for i, (o, n) in enumerate(zip(offs, nums)):
            oracle_update(int(o), int(n), g_np, float(r["h"][i]), t, step_ties)
        check_decisions(opt.get_stats(), opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        if teacher_forced or t == n_steps:
            compare(t, step_ties)
        rep.steps = t
    st = opt.get_stats()
    assert st["steps_done"] == n_steps and np.array_equal(st["clip_count"], clip_count) and st["status"] == 0
    for a, name in ((theta, "theta"), (m, "m"), (v, "v")):
        assert bool((a[pad_mask].float() == GUARD).all()), f"guard bands between tensors were overwritten in {name}"
    if optimizer == "lion":
        assert int((sign_ties > 0).sum()) <= 1e-3 * wl.n_params + 50
    opt.close()
    return rep


def run_sampled_bf16_state(wl: workloads.Workload, n_steps: int, device="cuda", k: int = 2048,
                           hyper_over: Optional[dict] = None, stochastic_seed: Optional[int] = None) -> ParityReport:
    """Full-size layouts with bfloat16 moments: all norms / decisions / gamma against the oracle, and theta, m, v on
    sampled elements that the oracle follows one by one (free-running; m and v bit-identical, theta within tolerance)."""
    hp = hyper_of(wl, **(hyper_over or {}))
    offs = np.array([t.offset for t in wl.tensors], np.int64)
    nums = np.array([t.numel for t in wl.tensors], np.int64)
    opt = binding.AdaGC(nums.tolist(), offs.tolist(), wl.torch_grad_dtype, hp["lambda_abs"], device=device,
                        state_dtype=torch.bfloat16)
    if stochastic_seed is not None:
        opt.set_state_rounding(True, stochastic_seed)
    rng = np.random.RandomState(99)
    samp = [sample_indices(int(n), k, rng) + int(o) for o, n in zip(offs, nums)]
    sizes = np.array([len(s) for s in samp], np.int64)
    soff = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.int64)
    flat_np = np.ascontiguousarray(np.concatenate(samp), dtype=np.int64)
    flat = torch.from_numpy(flat_np).to(device)
    rep = ParityReport()
    gamma = np.zeros(wl.n_tensors, np.float32)
    clip_count = np.zeros(wl.n_tensors, np.uint64)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device=device)
    theta = workloads.init_params(wl, device)
    m = torch.zeros(wl.arena_elems, dtype=torch.bfloat16, device=device)
    v = torch.zeros_like(m)
    s_theta = theta[flat].cpu().numpy().copy()
    s_m, s_v = np.zeros(len(flat_np), np.uint16), np.zeros(len(flat_np), np.uint16)
    for t in range(1, n_steps + 1):
        g = workloads.grads_for_step(wl, t, device)
        g_np = to_numpy_grads(g)
        s_g = np.ascontiguousarray(g_np[flat_np])
        opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"],
                 hp["beta"], hp["warmup"])
        ssq = c_oracle.sumsq_tensors(g_np, offs, nums)
        r = c_oracle.clip_decisions(ssq, gamma, t, hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"])
        clip_count += r["flag"].astype(np.uint64)
        check_decisions(opt.get_stats(), opt.get_sumsq(), ema.cpu().numpy(), r, rep, t)
        for i in range(wl.n_tensors):
            sl = slice(int(soff[i]), int(soff[i] + sizes[i]))
            c_oracle.adamw_update_bf16state(s_theta[sl], s_g[sl], s_m[sl], s_v[sl], float(r["h"][i]), t, hp["lr"],
                                            hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], fp32_decision=True,
                                            stochastic_seed=stochastic_seed, index=np.ascontiguousarray(flat_np[sl]))
        rep.steps = t
        del g
    st = opt.get_stats()
    assert st["steps_done"] == n_steps and np.array_equal(st["clip_count"], clip_count) and st["status"] == 0
    g_theta = theta[flat].cpu().numpy()
    g_m, g_v = _bf16_view(m[flat]), _bf16_view(v[flat])
    for i, t_ in enumerate(wl.tensors):
        sl = slice(int(soff[i]), int(soff[i] + sizes[i]))
        _assert_same_bf16("m", g_m[sl], s_m[sl], t_.name)
        _assert_same_bf16("v", g_v[sl], s_v[sl], t_.name)
        check_state("theta", g_theta[sl], s_theta[sl], rep, t_.name)
    opt.close()
    return rep
