"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Bar: clip flags / clip counts / step counter bit-exact; norms, gamma, h within 1e-5 relative;
fp32 theta, m, v within 1e-5 (per-tensor L2 and per element); bf16 clipped gradients within one ulp.
"""
import numpy as np
import pytest
import torch

from paper_2502_11034_b200 import binding, workloads

import parity_harness as H

pytestmark = pytest.mark.gpu


def _report(name, rep):
    print(f"\n[parity] {name}: {rep.line()}")


# ------------------------------------------------------------------ the five configurations
def test_tiny_all_elements():
    """Config 1: 8 fp32 tensors, 12 steps, x100 spike on tensor index 3 at step 6."""
    wl = workloads.build("tiny")
    rep = H.run_full(wl, wl.n_steps)
    _report("tiny", rep)
    assert rep.clipped > 0
    # lambda_abs = 1 never clips this layout in warm-up; a smaller threshold exercises that branch
    rep2 = H.run_full(wl, wl.n_steps, hyper_over=dict(lambda_abs=0.5))
    _report("tiny lambda_abs=0.5", rep2)
    # the 1-based reading of "tensor 3"
    wl.extra["spike_tensor"] = 2
    _report("tiny spike on index 2", H.run_full(wl, wl.n_steps))


def test_gpt2_small_all_elements():
    """Config 2: 148 tensors, bf16 gradients with per-tensor scales, 50 steps, 1% spiked x50 per step."""
    wl = workloads.build("gpt2_small")
    rep = H.run_full(wl, wl.n_steps)
    _report("gpt2_small", rep)
    assert rep.decisions == 148 * 50 and rep.clipped > 0
    # with lambda_abs = 1 the warm-up clips hard and seeds gamma low, so every later decision is a clip
    # with a wide margin; a large lambda_abs gives the mixed, close decisions that test bit-exactness
    rep = H.run_full(wl, 30, hyper_over=dict(lambda_abs=1e4))
    _report("gpt2_small lambda_abs=1e4", rep)
    assert 0 < rep.clipped < rep.decisions


def test_many_small_all_elements():
    """Config 4: 20 000 fp32 tensors, Student-t(2) gradients, 30 steps."""
    wl = workloads.build("many_small")
    rep = H.run_full(wl, wl.n_steps)
    _report("many_small", rep)
    assert rep.decisions == 20000 * 30 and rep.clipped > 0
    rep = H.run_full(wl, 20, hyper_over=dict(lambda_abs=1e4))
    _report("many_small lambda_abs=1e4", rep)
    assert 0 < rep.clipped < rep.decisions


def test_llama32_1b_sampled_adamw_and_clip_only():
    """Config 5 at full size: all decisions for 100 steps; state / clipped gradients on samples."""
    wl = workloads.build("llama32_1b")
    rep = H.run_sampled(wl, wl.n_steps, mode="adamw")
    _report("llama32_1b adamw", rep)
    assert rep.decisions == 146 * 100 and rep.clipped > 0
    rep = H.run_sampled(wl, 30, mode="clip", in_place=True)
    _report("llama32_1b clip-only in place", rep)
    rep = H.run_sampled(wl, 14, mode="clip", in_place=False)
    _report("llama32_1b clip-only out of place", rep)


def test_llama2_7b_sampled():
    """Config 3 at full size (the benchmark's launch configuration): 20 steps, spike at step 12."""
    free, _ = torch.cuda.mem_get_info()
    wl = workloads.build("llama2_7b")
    need = wl.arena_elems * 14 + (4 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    rep = H.run_sampled(wl, wl.n_steps, mode="adamw", k=1024)
    _report("llama2_7b", rep)
    assert rep.decisions == 291 * 20
    assert rep.clipped >= 8
    # With lambda_abs = 1 the warm-up clips (global norm 8.2) and every later decision is a clip; with a large
    # lambda_abs the steady state is calm and exactly the eight spiked tensors are clipped at step 12.
    rep = H.run_sampled(wl, 13, mode="adamw", k=256, hyper_over=dict(lambda_abs=1e4))
    _report("llama2_7b lambda_abs=1e4", rep)
    assert 8 <= rep.clipped < 291


def test_one_tensor_beyond_2_to_32_elements():
    """Maximum sizes: a single tensor of 2^32 + 12345 elements (262 145 chunks, element indices that do not fit
    32 bits) followed by a small tensor whose offset lies beyond 2^32.  All norms and decisions against the
    oracle (it streams the whole gradient), state on sampled elements including both ends and the last chunk."""
    n_big = 2 ** 32 + 12345
    specs, total = workloads._layout([("big", (n_big,)), ("small", (1000,))])
    free, _ = torch.cuda.mem_get_info()
    need = total * 14 + (6 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    hp = dict(workloads.PAPER_DEFAULTS, lambda_abs=1e4)
    wl = workloads.Workload("one_huge_tensor", 8, specs, "bf16", hp, warmup=1, n_steps=3, arena_elems=total,
                            grad_kind="normal", grad_scale=1e-4,
                            extra={"spike_step": 3, "spike_tensor": 1, "spike_factor": 40.0})
    assert specs[1].offset > 2 ** 32
    rep = H.run_sampled(wl, 3, mode="adamw", k=4096)
    _report("one tensor of 2^32 + 12345 elements", rep)
    assert rep.decisions == 6 and rep.clipped >= 1


def test_hand_worked_example_on_the_gpu():
    """The 2-tensor worked example (tests/golden/worked_example.json): every norm, clip factor, flag and gamma
    of the table is exactly representable, so the CUDA path must reproduce the table exactly."""
    import json
    import os
    from oracle import adagc_oracle as npo
    gold = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_example.json")))
    hp = gold["hyper"]
    offs, nums = [0, 8], [2, 3]
    opt = binding.AdaGC(nums, offs, torch.float32, hp["lambda_abs"])
    theta = torch.zeros(16, device="cuda")
    theta[0:2] = torch.tensor(gold["theta0"]["A"])
    theta[8:11] = torch.tensor(gold["theta0"]["B"])
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(2, device="cuda")
    ref = npo.AdaGCAdamW([gold["theta0"]["A"], gold["theta0"]["B"]], npo.Hyper(**hp), np.float32)
    for srow in gold["steps"]:
        g = torch.zeros(16, device="cuda")
        g[0:2] = torch.tensor(srow["gA"])
        g[8:11] = torch.tensor(srow["gB"])
        opt.step(theta, g, m, v, ema, srow["t"], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                 hp["lambda_rel"], hp["beta"], hp["warmup"])
        ref.step([np.array(srow["gA"], np.float32), np.array(srow["gB"], np.float32)])
        st = opt.get_stats()
        assert st["norm"].tolist() == srow["norm"] and st["h"].tolist() == srow["h"]
        assert st["flag"].astype(int).tolist() == srow["flag"] and ema.cpu().tolist() == srow["gamma"]
    th = theta.cpu().numpy()
    np.testing.assert_allclose(th[0:2], ref.theta[0], rtol=1e-5)
    np.testing.assert_allclose(th[8:11], ref.theta[1], rtol=1e-5)
    assert float(theta[2:8].abs().sum()) == 0.0 and st["clip_count"].tolist() == [3, 1]
    opt.close()


# ------------------------------------------------------------------ small layouts, all elements
@pytest.mark.parametrize("name,over", [
    ("llama2_7b", dict(n_layer=2, d=256, ffn=688, vocab=1000)),
    ("llama32_1b", dict(n_layer=2, d=128, ffn=512, vocab=2000, kv_dim=32)),
    ("gpt2_small", dict(n_layer=2, d=96, vocab=1031, n_pos=64)),
    ("many_small", dict(n_tensors=300, lo=1, hi=40000)),
])
def test_small_layouts_all_elements(name, over):
    wl = workloads.build(name, **over)
    rep = H.run_full(wl, min(wl.n_steps, 25))
    _report(f"{name} (small)", rep)
    # both kernels of the update phase, forced
    for path in (binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK):
        rep = H.run_full(wl, 8, flags=path)
        _report(f"{name} (small, update path {path})", rep)


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
def test_lion_small_layouts_all_elements(path):
    """The clip fused with Lion (Section 4.2: optimizer-agnostic use), both update kernels."""
    for name, over in [("llama2_7b", dict(n_layer=2, d=256, ffn=688, vocab=1000)),
                       ("many_small", dict(n_tensors=300, lo=1, hi=40000))]:
        wl = workloads.build(name, **over)
        rep = H.run_full_lion(wl, 15, flags=path)
        _report(f"lion {name} (small, path {path})", rep)


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
def test_sgdm_small_layouts_all_elements(path):
    """The clip fused with SGD with momentum, both update kernels, both gradient dtypes."""
    for name, over in [("llama2_7b", dict(n_layer=2, d=256, ffn=688, vocab=1000)),
                       ("many_small", dict(n_tensors=300, lo=1, hi=40000))]:
        wl = workloads.build(name, **over)
        rep = H.run_full_sgdm(wl, 15, flags=path, hyper_over=dict(lambda_abs=1e4))
        _report(f"sgdm {name} (small, path {path})", rep)
        assert rep.clipped > 0


def test_lion_gpt2_small_all_elements():
    wl = workloads.build("gpt2_small")
    rep = H.run_full_lion(wl, 20, hyper_over=dict(lambda_abs=1e4))
    _report("lion gpt2_small", rep)
    assert 0 < rep.clipped < rep.decisions


@pytest.mark.parametrize("in_place", [True, False], ids=["in_place", "out_of_place"])
def test_clip_only_small_layouts_all_elements(in_place):
    """adagc_clip on every element, both gradient dtypes; calm and spiky steady states."""
    for name, over, hov in [("llama32_1b", dict(n_layer=2, d=128, ffn=512, vocab=2000, kv_dim=32), dict(lambda_abs=1e4)),
                            ("many_small", dict(n_tensors=300, lo=1, hi=40000), dict(lambda_abs=1e4)),
                            ("tiny", {}, {})]:
        wl = workloads.build(name, **over)
        rep = H.run_full_clip(wl, 12, in_place, hyper_over=hov)
        _report(f"clip-only {name} in_place={in_place}", rep)
        assert rep.clipped > 0


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
@pytest.mark.parametrize("in_place", [True, False], ids=["in_place", "out_of_place"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_clip_only_ragged(dtype, in_place, path):
    """The clip-only entry on a ragged layout, in contexts of either update path: full and partial chunks, ragged tails,
    tensors that are skipped in place because h == 1 between tensors that are not; padding between tensors must stay
    untouched out of place."""
    sizes = [1, 7, 8, 9, 255, 2049, 16383, 16384, 16385, 3 * 16384 + 5, 100003, 40 * 16384, 9 * 16384 + 4095, 6 * 16384,
             16384, 5 * 16384 + 8]
    wl = _ragged_workload(sizes, dtype)
    rep = H.run_full_clip(wl, 8, in_place, flags=path, hyper_over=dict(lambda_abs=1e4, warmup=2))
    _report(f"clip-only ragged {dtype} in_place={in_place} path {path}", rep)
    assert 0 < rep.clipped < rep.decisions            # some tensors clipped, some passed through


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
def test_emit_bf16_parameters_all_elements(path):
    """adagc_step_emit_bf16: fp32 master parameters plus the bf16 working copy from the same kernel."""
    sizes = [1, 7, 8, 9, 255, 2049, 16384, 16385, 3 * 16384 + 5, 40 * 16384, 100003]
    for dtype in ("bf16", "f32"):
        rep = H.run_full(_ragged_workload(sizes, dtype), 6, flags=path, emit_bf16=True)
        _report(f"emit bf16, {dtype} grads, path {path}", rep)
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    _report(f"emit bf16 llama (small), path {path}", H.run_full(wl, 12, flags=path, emit_bf16=True))
    # an fp32-gradient layout whose offsets are multiples of 4 but not of 8 cannot carry a bf16 arena
    opt = binding.AdaGC([100, 60], [0, 100], torch.float32, 1.0, flags=path)
    z = torch.zeros(160, device="cuda")
    with pytest.raises(binding.AdagcError) as e:
        opt.step_emit_bf16(z, torch.zeros(160, device="cuda", dtype=torch.bfloat16), z.clone(), z.clone(), z.clone(),
                           torch.zeros(2, device="cuda"), 1, 1e-3, 0.9, 0.95, 1e-8, 0.1, 1.04, 0.99, 0)
    assert e.value.status == -2
    opt.close()


def test_moe_layout_small_all_elements():
    """Mixture-of-experts tensor census ((7+3E)L+3 tensors, Section 4.3 "Memory"), reduced dimensions."""
    wl = workloads.build("moe_8x1b", n_layer=2, d=128, ffn=352, vocab=1000, kv_dim=32, n_experts=4)
    assert wl.n_tensors == (7 + 3 * 4) * 2 + 3
    rep = H.run_full(wl, 20, hyper_over=dict(lambda_abs=1e4))
    _report("moe (small)", rep)
    assert 0 < rep.clipped < rep.decisions


def test_ernie_moe_layout_small_all_elements():
    """The fine-grained MoE census the paper prints ((9+3E)L+3 tensors, Section 4.3 "Memory"), reduced dimensions."""
    wl = workloads.build("moe_ernie", n_layer=2, d=160, ffn=64, vocab=1000, kv_dim=32, n_experts=6)
    assert wl.n_tensors == (9 + 3 * 6) * 2 + 3
    rep = H.run_full(wl, 20, hyper_over=dict(lambda_abs=1e4))
    _report("ernie moe (small)", rep)
    assert 0 < rep.clipped < rep.decisions


@pytest.mark.parametrize("variant", ["keep_initial", "global_adaptive", "both"])
def test_ablation_variants_all_elements(variant):
    """Section 5 variants: caller-given gamma_0 (no seeding at t = 1) and Global AdaGC (one adaptive threshold)."""
    flags = {"keep_initial": binding.EMA_KEEP_INITIAL, "global_adaptive": binding.CLIP_GLOBAL_ADAPTIVE,
             "both": binding.EMA_KEEP_INITIAL | binding.CLIP_GLOBAL_ADAPTIVE}[variant]
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    for warmup, gamma0 in ((0, 0.02), (3, 0.5)):
        rep = H.run_full(wl, 16, flags=flags, gamma0=gamma0, hyper_over=dict(warmup=warmup, lambda_abs=1e4))
        _report(f"{variant} warmup={warmup} gamma0={gamma0}", rep)
    assert rep.steps == 16


def test_thresholded_initialization_all_elements():
    """Section 5, EMA-initialization variant 3: gamma = min(clipped norm, cap) at seeding and in warm-up."""
    wl = workloads.build("llama2_7b", n_layer=2, d=256, ffn=688, vocab=1000)
    for warmup, cap, flags in ((4, 0.01, 0), (0, 0.005, 0), (3, 0.02, binding.CLIP_GLOBAL_ADAPTIVE)):
        rep = H.run_full(wl, 14, flags=flags, ema_cap=cap, hyper_over=dict(warmup=warmup, lambda_abs=1e4))
        _report(f"thresholded init warmup={warmup} cap={cap} flags={flags}", rep)
        assert rep.clipped > 0
    wl = workloads.build("many_small", n_tensors=300, lo=1, hi=40000)
    rep = H.run_full(wl, 12, ema_cap=0.1, hyper_over=dict(lambda_abs=1e4))          # the paper's cap
    _report("thresholded init many_small cap=0.1", rep)
    opt = binding.AdaGC([8], [0], torch.float32, 1.0)
    for bad in (-1.0, float("nan"), float("inf")):
        with pytest.raises(binding.AdagcError):
            opt.set_ema_cap(bad)
    opt.close()


def _ragged_workload(sizes, dtype):
    specs, total = workloads._layout([(f"t{i}", (n,)) for i, n in enumerate(sizes)])
    hp = dict(workloads.PAPER_DEFAULTS, lambda_abs=0.05)
    return workloads.Workload("ragged", 7, specs, dtype, hp, warmup=2, n_steps=8, arena_elems=total,
                              grad_kind="student_t", grad_df=3, grad_scale=1e-3,
                              extra={"spike_frac": 0.2, "spike_lo": 5.0, "spike_hi": 500.0})


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_tails_and_chunk_edges(dtype, path):
    """Sizes around the vector width and the 16384-element chunk: tails of 1..7 elements,
    one element short of / past a chunk, several chunks plus a tail."""
    sizes = [1, 2, 3, 5, 7, 8, 9, 10, 15, 16, 17, 31, 33, 255, 257, 2047, 2049, 16383, 16384, 16385,
             32767, 32768, 32769, 3 * 16384 + 5, 100003, 40 * 16384, 9 * 16384 + 4095]
    rep = H.run_full(_ragged_workload(sizes, dtype), 8, flags=path)
    _report(f"ragged {dtype} path {path}", rep)
    assert rep.clipped > 0


@pytest.mark.parametrize("seed", range(10))
def test_random_layouts(seed):
    """Seeded random layouts: tensor count, sizes (log-uniform, so tails, single chunks and multi-chunk tensors
    mix), gradient dtype, update kernel, warm-up length, thresholds and entry point all drawn at random."""
    rng = np.random.RandomState(1000 + seed)
    n_t = int(rng.randint(1, 60))
    sizes = np.unique(np.round(np.exp(rng.uniform(0.0, np.log(300000.0), size=n_t))).astype(np.int64)).tolist()
    rng.shuffle(sizes)
    dtype = ["f32", "bf16"][int(rng.randint(2))]
    flags = [0, binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK, binding.FUSED_SMALL][int(rng.randint(4))]
    if flags != binding.FUSED_SMALL:      # where the decisions are taken: norm kernel's tail (default) or a kernel of their own
        flags |= [0, binding.SEPARATE_FINALIZE][int(rng.randint(2))]
    over = dict(warmup=int(rng.randint(0, 4)), lambda_abs=float(np.exp(rng.uniform(np.log(1e-3), np.log(1e2)))),
                lambda_rel=float(rng.uniform(1.0, 1.3)), beta=float(rng.uniform(0.5, 0.999)))
    wl = _ragged_workload(sizes, dtype)
    how = ["", "", "eager", "graph"][int(rng.randint(4))] if flags != binding.FUSED_SMALL else ""
    rep = H.run_full(wl, 7, flags=flags, hyper_over=over, capturable=how)
    _report(f"random layout {seed}: T={len(sizes)} {dtype} flags={flags} {over} capturable={how!r}", rep)


@pytest.mark.parametrize("where", [0, binding.SEPARATE_FINALIZE], ids=["norm_tail", "own_kernel"])
def test_decisions_in_the_norm_tail_and_in_their_own_kernel(where):
    """Both places where an AdaGC step can take its per-tensor decisions, forced, on layouts that exercise what differs
    between them: tensors inside one block's range of chunks, tensors shared by many blocks (tickets), a tensor with
    more than 1024 chunks (summed by a whole block), thousands of one-chunk tensors."""
    sizes = [1, 9, 300, 16384, 16385, 5 * 16384 + 3, 1100 * 16384 + 77, 40 * 16384, 2049, 70000]
    for dtype in ("f32", "bf16"):
        _report(f"decisions flag {where} {dtype}", H.run_full(_ragged_workload(sizes, dtype), 6, flags=where))
    wl = workloads.build("many_small", n_tensors=5000, lo=16, hi=40000)
    _report(f"decisions flag {where}, 5000 tensors", H.run_full(wl, 8, flags=where, hyper_over=dict(lambda_abs=1e4)))
    a, _ = _run_gpu(*_mini(), 8, flags=where)
    b, _ = _run_gpu(*_mini(), 8, flags=binding.SEPARATE_FINALIZE - where)
    for x, y in zip(a, b):
        assert torch.equal(x, y)                                   # bit-identical wherever the decisions are taken


def test_launch_grids_match_the_residency_the_kernels_are_tuned_for():
    """Eight resident 256-thread blocks per SM for the norm / scale kernels, one block per SM for the bulk-async update
    kernel and two for the register one: a kernel whose register count stops admitting that (the occupancy query at
    adagc_create then sizes a smaller grid) shows here, not only in a timing."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    wl = workloads.build("gpt2_small", n_layer=4, d=768, vocab=4096, n_pos=64)      # about two thousand chunks
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    for state in (torch.float32, torch.bfloat16):
        for flags, per_sm in ((binding.UPDATE_PATH_BULK, 1), (binding.UPDATE_PATH_REGISTERS, 2), (0, 1)):
            opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, 1.0, flags=flags, state_dtype=state)
            assert opt.launch_grids() == (8 * sms, per_sm * sms)
            opt.close()
    small = binding.AdaGC([100, 20000], [0, 104], torch.float32, 1.0)              # three chunks: one block each
    assert small.launch_grids() == (3, 3)
    small.close()
    assert binding.lib().adagc_launch_grids(None, None, None) == -1


def test_single_tensor_and_warmup_zero():
    """T = 1 (the 'global adaptive' view) and T_start = 0 (gamma seeded from the first norm)."""
    wl = _ragged_workload([50000], "bf16")
    _report("T=1", H.run_full(wl, 6))
    wl = _ragged_workload([40, 5000, 70000], "f32")
    _report("warmup=0", H.run_full(wl, 8, hyper_over=dict(warmup=0)))
    _report("always warm-up", H.run_full(wl, 5, hyper_over=dict(warmup=100, lambda_abs=1e-3)))
    _report("eps=1e-15, beta2=0.999, lr schedule",
            H.run_full(wl, 8, hyper_over=dict(eps=1e-15, beta2=0.999), lr_schedule=lambda t: 1e-3 * t / 8))


# ------------------------------------------------------------------ properties and edge cases
def _mini():
    wl = workloads.build("llama2_7b", n_layer=1, d=128, ffn=344, vocab=500)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    return wl, offs, nums


def _run_gpu(wl, offs, nums, steps, start_state=None, first_step=1, flags=0):
    hp = H.hyper_of(wl)
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], flags=flags)
    if start_state is None:
        theta = workloads.init_params(wl, "cuda")
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device="cuda")
    else:
        theta, m, v, ema = (a.clone() for a in start_state)
    flags = []
    for t in range(first_step, first_step + steps):
        g = workloads.grads_for_step(wl, t, "cuda")
        opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                 hp["lambda_rel"], hp["beta"], hp["warmup"])
        flags.append(opt.get_stats()["flag"].copy())
    opt.close()
    return (theta, m, v, ema), flags


def test_run_twice_is_bit_identical():
    wl, offs, nums = _mini()
    a, fa = _run_gpu(wl, offs, nums, 12)
    b, fb = _run_gpu(wl, offs, nums, 12)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert all(np.array_equal(p, q) for p, q in zip(fa, fb))


def test_checkpoint_resume_is_bit_identical():
    """The caller's buffers (theta, m, v, gamma) and the step number are the whole state."""
    wl, offs, nums = _mini()
    full, _ = _run_gpu(wl, offs, nums, 16)
    half, _ = _run_gpu(wl, offs, nums, 8)
    saved = tuple(a.cpu() for a in half)                        # "checkpoint"
    resumed, _ = _run_gpu(wl, offs, nums, 8, start_state=tuple(a.cuda() for a in saved), first_step=9)
    for x, y in zip(full, resumed):
        assert torch.equal(x, y)


def test_zero_and_nonfinite_gradients_and_absorbing_gamma():
    from oracle import c_oracle
    nums, offs = [1000, 24, 3000], [0, 1000, 1024]
    opt = binding.AdaGC(nums, offs, torch.float32, 1.0)
    theta = torch.randn(4024, device="cuda", generator=torch.Generator("cuda").manual_seed(5))
    theta0 = theta.cpu().numpy().copy()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(3, dtype=torch.float32, device="cuda")
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1, lambda_rel=1.04, beta=0.9, lambda_abs=1.0, warmup=0)
    ref = c_oracle.ArenaOracle(offs, nums, theta0, **hp)
    gen = torch.Generator("cuda").manual_seed(6)
    for t in range(1, 7):
        g = torch.randn(4024, device="cuda", generator=gen) * 1e-2
        if t == 1:
            g[1000:1024] = 0.0                                  # gamma of tensor 1 seeded with 0 ...
        if t in (3, 4):
            g[0:1000] = 0.0                                     # zero gradient: no clip, gamma decays
        if t == 5:
            g[1024 + 17] = float("inf")
        if t == 6:
            g[1024 + 5] = float("nan")
        opt.step(theta, g, m, v, ema, t, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                 hp["lambda_rel"], hp["beta"], hp["warmup"])
        r = ref.step(g.cpu().numpy())
        st = opt.get_stats()
        assert np.array_equal(st["flag"], r["flag"]), f"step {t}"
        got, want = ema.cpu().numpy(), r["gamma"]
        assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(np.isinf(got), np.isinf(want))
        fin = np.isfinite(want)
        np.testing.assert_allclose(got[fin], want[fin], rtol=1e-5)
        if t >= 2:
            assert st["flag"][1] and st["h"][1] == 0.0 and got[1] == 0.0      # ... is absorbing
        assert (st["status"] & binding.ADAGC_W_NONFINITE) == (binding.ADAGC_W_NONFINITE if t >= 5 else 0)
    th = theta.cpu().numpy()
    bad = np.isnan(ref.theta)
    assert np.array_equal(np.isnan(th), bad)                     # NaN propagates as in plain AdamW ...
    assert set(np.nonzero(bad)[0]) == {1024 + 17, 1024 + 5}      # ... and only where the gradient was bad
    np.testing.assert_allclose(th[~bad], ref.theta[~bad], rtol=1e-5, atol=1e-7)
    opt.close()


def test_argument_errors_enqueue_nothing():
    nums, offs = [100, 60], [0, 104]
    opt = binding.AdaGC(nums, offs, torch.bfloat16, 1.0)
    theta = torch.ones(164, device="cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    g = torch.ones(164, device="cuda", dtype=torch.bfloat16)
    ema = torch.zeros(2, device="cuda")
    ok = dict(step=1, lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1, lambda_rel=1.04, beta=0.99, warmup=0)
    for bad in (dict(step=0), dict(beta=1.0), dict(beta=-0.1), dict(lambda_rel=0.0), dict(beta1=1.0),
                dict(eps=-1.0), dict(warmup=-1), dict(lr=float("nan"))):
        kw = dict(ok, **bad)
        with pytest.raises(binding.AdagcError) as e:
            opt.step(theta, g, m, v, ema, **kw)
        assert e.value.status == -1
    with pytest.raises(binding.AdagcError) as e:
        opt.step(theta[1:], g, m, v, ema, **ok)                   # misaligned arena pointer
    assert e.value.status == -2
    torch.cuda.synchronize()
    assert opt.launch_count() == 0 and bool((theta == 1).all()) and opt.get_stats()["steps_done"] == 0
    opt.close()


def test_bounded_wait_gives_up_and_context_stays_usable():
    """A device-side wait that is never satisfied runs out after its limit, reports ADAGC_E_TIMEOUT through
    the status word, and the same context then runs a correct step (nothing faults, nothing hangs)."""
    import time
    wl, offs, nums = _mini()
    hp = H.hyper_of(wl)
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], flags=binding.UPDATE_PATH_BULK)
    assert opt.get_stats()["status"] == 0
    t0 = time.perf_counter()
    opt.debug_wait_timeout(50.0)
    st = opt.get_stats()                                           # synchronises
    dt = time.perf_counter() - t0
    assert st["status"] & binding.ADAGC_E_TIMEOUT and 0.04 < dt < 5.0
    theta = workloads.init_params(wl, "cuda")
    before = theta.clone()
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device="cuda")
    g = workloads.grads_for_step(wl, 1, "cuda")
    opt.step(theta, g, m, v, ema, 1, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
             hp["lambda_rel"], hp["beta"], hp["warmup"])
    st = opt.get_stats()
    assert st["steps_done"] == 1 and np.isfinite(st["norm"]).all() and not torch.equal(theta, before)
    opt.close()


def test_one_kernel_step_refuses_work_after_a_timed_out_barrier_was_seen():
    """After a grid barrier of the one-kernel step has timed out, the device-side arrival counter and the host's
    barrier count differ for good.  The host latches the ADAGC_E_TIMEOUT bit when it reads the status word and refuses
    later steps of that context.  The bit is fed to the latch by hand here: no barrier is made to time out on the GPU."""
    wl, offs, nums = _mini()
    hp = H.hyper_of(wl)
    args = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    theta = workloads.init_params(wl, "cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device="cuda")
    g = workloads.grads_for_step(wl, 1, "cuda")
    fused = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], flags=binding.FUSED_SMALL)
    plain = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
    fused.step(theta, g, m, v, ema, 1, *args)
    fused.debug_latch_status(binding.ADAGC_W_NONFINITE)            # other bits do not poison the context
    fused.step(theta, g, m, v, ema, 2, *args)
    assert fused.get_stats()["steps_done"] == 2
    before = theta.clone()
    fused.debug_latch_status(binding.ADAGC_E_TIMEOUT)
    with pytest.raises(binding.AdagcError) as e:
        fused.step(theta, g, m, v, ema, 3, *args)
    assert e.value.status == -9 and "anew" in binding.strerror(-9)
    torch.cuda.synchronize()
    assert torch.equal(theta, before) and fused.get_stats()["steps_done"] == 2     # nothing was enqueued
    plain.debug_latch_status(binding.ADAGC_E_TIMEOUT)              # the three-launch step has no such state
    plain.step(theta, g, m, v, ema, 1, *args)
    fused.close()
    plain.close()


def test_phase_timing_and_launch_count():
    wl, offs, nums = _mini()
    hp = H.hyper_of(wl)
    opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
    theta = workloads.init_params(wl, "cuda")
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device="cuda")
    g = workloads.grads_for_step(wl, 1, "cuda")
    opt.set_phase_timing(True)
    args = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"])
    opt.step(theta, g, m, v, ema, 1, *args, 1)                    # warm-up step: 4 kernels
    assert opt.launch_count() == 4
    opt.step(theta, g, m, v, ema, 2, *args, 1)                    # AdaGC step: 2 kernels (the decisions are taken in the
    assert opt.launch_count() == 6                                # norm kernel's tail)
    ms = opt.get_phase_times()
    assert len(ms) == 3 and all(x >= 0 for x in ms)
    opt.close()


@pytest.mark.parametrize("layout", ["mini", "gpt2_small"])
@pytest.mark.parametrize("state", [torch.float32, torch.bfloat16], ids=["fp32_state", "bf16_state"])
def test_step_host_matches_device_entry(layout, state):
    """The host-buffer entry gives bit-identical results; on the larger layout (several groups of tensors)
    its AdaGC steps run pipelined behind the host-to-device copies, its warm-up steps do not."""
    if layout == "mini":
        wl, offs, nums = _mini()
    else:
        wl = workloads.build("gpt2_small")
        wl.warmup = 3
        offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    hp = H.hyper_of(wl, lambda_abs=1e4)
    args = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    outs = []
    for host in (False, True):
        opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], state_dtype=state)
        theta = workloads.init_params(wl, "cuda")
        m = torch.zeros(wl.arena_elems, dtype=state, device="cuda")
        v = torch.zeros_like(m)
        ema = torch.zeros(wl.n_tensors, dtype=torch.float32, device="cuda")
        g_dev = torch.empty(wl.arena_elems, dtype=wl.torch_grad_dtype, device="cuda")
        norm = torch.empty(wl.n_tensors, dtype=torch.float32).pin_memory()
        hfac = torch.empty(wl.n_tensors, dtype=torch.float32).pin_memory()
        flag = torch.empty(wl.n_tensors, dtype=torch.uint8).pin_memory()
        for t in range(1, 9):
            g = workloads.grads_for_step(wl, t, "cuda")
            if host:
                opt.step_host(theta, g_dev, m, v, ema, g.cpu().pin_memory(), t, *args, norm, hfac, flag)
                st = opt.get_stats()
                assert np.array_equal(norm.numpy(), st["norm"]) and np.array_equal(flag.numpy().astype(bool), st["flag"])
                assert np.array_equal(hfac.numpy(), st["h"])
            else:
                opt.step(theta, g, m, v, ema, t, *args)
        final = opt.get_stats()
        assert final["steps_done"] == 8 and final["status"] == 0
        outs.append((theta, m, v, ema, torch.from_numpy(final["clip_count"].astype(np.int64))))
        opt.close()
    for x, y in zip(*outs):
        assert torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x,
                           y.view(torch.int16) if y.dtype == torch.bfloat16 else y)
    assert int(outs[0][4].sum()) > 0
