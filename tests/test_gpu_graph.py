"""The capturable step (adagc_step_capturable): step number, warm-up switch, gamma seeding and bias corrections
derived on the device, so one captured CUDA graph serves every step.  Parity bar as for adagc_step: decisions
and counters bit-exact, norms / gamma / h / fp32 state within 1e-5 of the CPU oracle."""
import time

import numpy as np
import pytest
import torch

from paper_2502_11034_b200 import binding, workloads

import parity_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("how", ["eager", "graph"])
def test_capturable_step_matches_the_oracle(how):
    wl = workloads.build("tiny")
    rep = H.run_full(wl, wl.n_steps, capturable=how)
    print(f"\n[parity] capturable {how} tiny: {rep.line()}")
    assert rep.clipped > 0
    rep = H.run_full(wl, wl.n_steps, capturable=how, hyper_over=dict(lambda_abs=0.5, warmup=0))
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    for flags in (0, binding.UPDATE_PATH_REGISTERS, binding.CLIP_GLOBAL_ADAPTIVE):
        rep = H.run_full(wl, 14, capturable=how, flags=flags, hyper_over=dict(lambda_abs=1e4, warmup=4),
                         lr_schedule=lambda t: 3e-4 * min(1.0, t / 6))
        print(f"[parity] capturable {how} llama (small) flags={flags}: {rep.line()}")
        assert rep.clipped > 0
    wl = workloads.build("many_small", n_tensors=300, lo=1, hi=40000)
    rep = H.run_full(wl, 10, capturable=how, hyper_over=dict(lambda_abs=1e4), ema_cap=0.1)
    assert rep.steps == 10


def test_capturable_equals_plain_step_and_resumes_from_a_set_counter():
    """Same inputs through adagc_step and adagc_step_capturable: state within a few fp32 ulps (bit-identical unless
    the device's and the host's beta^t round to different fp32 coefficients); a run cut in two, with the counter
    restored by adagc_set_step_counter, is bit-identical to the uninterrupted capturable run."""
    wl = workloads.build("llama2_7b", n_layer=1, d=128, ffn=344, vocab=500)
    hp = H.hyper_of(wl, lambda_abs=1e4, warmup=3)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    a = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])

    def run(kind, steps, state=None, first=1):
        opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
        if state is None:
            theta = workloads.init_params(wl, "cuda")
            m, v = torch.zeros_like(theta), torch.zeros_like(theta)
            ema = torch.zeros(wl.n_tensors, device="cuda")
        else:
            theta, m, v, ema = (x.clone() for x in state)
            opt.set_step_counter(first - 1)
        for t in range(first, first + steps):
            g = workloads.grads_for_step(wl, t, "cuda")
            if kind == "plain":
                opt.step(theta, g, m, v, ema, t, *a)
            else:
                opt.step_capturable(theta, g, m, v, ema, *a)
        st = opt.get_stats()
        opt.close()
        return (theta, m, v, ema), st

    plain, st_p = run("plain", 12)
    cap, st_c = run("cap", 12)
    assert st_c["steps_done"] == 12 and np.array_equal(st_p["flag"], st_c["flag"])
    assert torch.equal(plain[3], cap[3])                              # gamma never depends on beta^t
    for x, y in zip(plain[:3], cap[:3]):
        assert torch.allclose(x, y, rtol=2e-6, atol=1e-12)
    half, _ = run("cap", 7)
    rest, st_r = run("cap", 5, state=half, first=8)
    assert st_r["steps_done"] == 12
    for x, y in zip(cap, rest):
        assert torch.equal(x, y)


def test_graph_replay_cuts_the_launch_cost_of_a_small_layout():
    """The tiny layout is bound by launch latency; replaying the captured step must not be slower than calling the
    three-launch entry point from the host, and the numbers are printed for the record."""
    wl = workloads.build("tiny")
    hp = H.hyper_of(wl)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
    theta = workloads.init_params(wl, "cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, device="cuda")
    g = workloads.grads_for_step(wl, 1, "cuda")
    a = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        opt.step_capturable(theta, g, m, v, ema, *a)
    K = 200

    def timed(fn):
        for _ in range(20):
            fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(K):
            fn()
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) / K * 1e6

    step = [opt.get_stats()["steps_done"]]

    def eager():
        step[0] += 1
        opt.step(theta, g, m, v, ema, step[0], *a)

    us_eager = timed(eager)
    us_graph = timed(graph.replay)
    print(f"\n[timing] tiny layout: adagc_step from the host {us_eager:.1f} us/step, graph replay of "
          f"adagc_step_capturable {us_graph:.1f} us/step")
    assert us_graph < 1.5 * us_eager
    assert opt.get_stats()["status"] == 0
    opt.close()


# ------------------------------------------------------------------ the one-kernel step for small layouts
def _ragged(sizes, dtype):
    specs, total = workloads._layout([(f"t{i}", (n,)) for i, n in enumerate(sizes)])
    hp = dict(workloads.PAPER_DEFAULTS, lambda_abs=0.05)
    return workloads.Workload("ragged", 7, specs, dtype, hp, warmup=2, n_steps=8, arena_elems=total,
                              grad_kind="student_t", grad_df=3, grad_scale=1e-3,
                              extra={"spike_frac": 0.2, "spike_lo": 5.0, "spike_hi": 500.0})


def test_fused_small_step_matches_the_oracle():
    """ADAGC_FUSED_SMALL: norm, decisions and AdamW in one cooperative kernel with grid barriers in between."""
    F = binding.FUSED_SMALL
    wl = workloads.build("tiny")
    rep = H.run_full(wl, wl.n_steps, flags=F)
    print(f"\n[parity] fused tiny: {rep.line()}")
    assert rep.clipped > 0
    H.run_full(wl, wl.n_steps, flags=F, hyper_over=dict(lambda_abs=0.5))                 # warm-up that clips
    H.run_full(wl, 8, flags=F, hyper_over=dict(warmup=0))
    sizes = [1, 7, 8, 9, 255, 2049, 16384, 16385, 3 * 16384 + 5, 100003, 40 * 16384]
    for dtype in ("f32", "bf16"):
        for path in (0, binding.UPDATE_PATH_REGISTERS):                                  # grids of one and two blocks per SM
            rep = H.run_full(_ragged(sizes, dtype), 8, flags=F | path)
            print(f"[parity] fused ragged {dtype} path {path}: {rep.line()}")
    wl = workloads.build("many_small", n_tensors=300, lo=1, hi=40000)
    rep = H.run_full(wl, 12, flags=F, hyper_over=dict(lambda_abs=1e4), ema_cap=0.1)
    assert 0 < rep.clipped < rep.decisions
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    rep = H.run_full(wl, 14, flags=F | binding.EMA_KEEP_INITIAL, gamma0=0.02, hyper_over=dict(warmup=0, lambda_abs=1e4))
    assert rep.steps == 14


def test_fused_small_limits_and_timing():
    """Too large a layout is refused at create; on the tiny layout the one-kernel step is timed against the
    three-launch step (printed for the record) and must not be slower."""
    with pytest.raises(binding.AdagcError) as e:
        binding.AdaGC([4097 * 16384], [0], torch.float32, 1.0, flags=binding.FUSED_SMALL)
    assert e.value.status == -1
    with pytest.raises(binding.AdagcError):
        binding.AdaGC([1000], [0], torch.float32, 1.0, flags=binding.FUSED_SMALL | binding.CLIP_GLOBAL_ADAPTIVE)
    wl = workloads.build("tiny")
    hp = H.hyper_of(wl)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    a = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    res = {}
    for name, flags in (("three launches", 0), ("one kernel", binding.FUSED_SMALL)):
        opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], flags=flags)
        theta = workloads.init_params(wl, "cuda")
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ema = torch.zeros(wl.n_tensors, device="cuda")
        g = workloads.grads_for_step(wl, 1, "cuda")
        t = 0
        for _ in range(30):
            t += 1
            opt.step(theta, g, m, v, ema, t, *a)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(300):
            t += 1
            opt.step(theta, g, m, v, ema, t, *a)
        torch.cuda.synchronize()
        res[name] = (time.perf_counter() - t0) / 300 * 1e6
        st = opt.get_stats()
        assert st["status"] == 0 and st["steps_done"] == t
        assert opt.launch_count() == (2 * t + 2 * hp["warmup"] if flags == 0 else t)   # AdaGC step: 2 kernels, warm-up step: 4
        opt.close()
    print(f"\n[timing] tiny layout, us per step: {res}")
    assert res["one kernel"] < 1.1 * res["three launches"]


def test_fused_small_with_tensors_the_rank_holds_nothing_of():
    """ADAGC_ALLOW_EMPTY tensors (no chunk at all) still get their statistics and their gamma decay in the one-kernel
    step; the result is bit-identical to the three-launch step on the same descriptor."""
    nums, offs = [100, 0, 5000, 0, 40000], [0, 0, 104, 0, 5104]
    total = 5104 + 40000
    a = (1e-3, 0.9, 0.95, 1e-8, 0.1, 1.04, 0.9, 2)
    res = []
    for flags in (binding.ALLOW_EMPTY, binding.ALLOW_EMPTY | binding.FUSED_SMALL):
        opt = binding.AdaGC(nums, offs, torch.float32, 0.01, flags=flags)
        gen = torch.Generator(device="cuda").manual_seed(5)
        theta = torch.randn(total, device="cuda", generator=gen) * 0.02
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ema = torch.full((5,), float("nan"), device="cuda")
        for t in range(1, 8):
            g = torch.randn(total, device="cuda", generator=gen) * (1e-3 if t != 5 else 0.1)
            opt.step(theta, g, m, v, ema, t, *a)
        st = opt.get_stats()
        res.append((theta.clone(), m.clone(), v.clone(), ema.clone(), st))
        opt.close()
    for x, y in zip(res[0][:4], res[1][:4]):
        assert torch.equal(x, y)
    for k in ("norm", "h", "flag", "clip_count"):
        assert np.array_equal(res[0][4][k], res[1][4][k])
    assert res[1][4]["steps_done"] == 7 and res[1][4]["status"] == 0
    assert res[1][4]["norm"][1] == 0.0 and float(res[1][3][1]) == 0.0          # empty tensor: norm 0, gamma decayed from 0
    assert res[0][4]["clip_count"].sum() > 0
