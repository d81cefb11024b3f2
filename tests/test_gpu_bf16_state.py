"""GPU parity with the optimizer moments stored as bfloat16 (adagc_desc.state_dtype = ADAGC_BF16): fp32 master theta,
bfloat16 m and v, fp32 arithmetic, theta updated from the unrounded moments, round-to-nearest-even where the moments
are stored.  The CUDA library is called through its C ABI and compared with the CPU oracle's bfloat16-state functions.

Bar: clip decisions, counters and gamma as everywhere else (bit-exact / 1e-5); theta within the fp32 tolerance; the
stored moments BIT-IDENTICAL to the oracle's on every element: which bfloat16 neighbour is stored is a discrete
decision that both sides take in single precision, in the operation order the library's header states.
"""
import numpy as np
import pytest
import torch

from paper_2502_11034_b200 import binding, workloads

import parity_harness as H
from test_gpu_parity import _ragged_workload, _report

pytestmark = pytest.mark.gpu

SEED = 0x5EED_0123_4567_89AB      # stochastic rounding of the stored moments

SIZES = [1, 2, 3, 5, 7, 8, 9, 10, 15, 16, 17, 31, 33, 255, 257, 2047, 2049, 4095, 4096, 4097, 16383, 16384, 16385,
         32767, 32768, 32769, 3 * 16384 + 5, 100003, 40 * 16384, 9 * 16384 + 4095]


@pytest.mark.parametrize("forced", [True, False], ids=["same_state_every_step", "free_running"])
def test_tiny_all_elements(forced):
    wl = workloads.build("tiny")
    rep = H.run_bf16_state(wl, wl.n_steps, teacher_forced=forced)
    _report(f"tiny, bf16 state, forced={forced}", rep)
    assert rep.clipped > 0


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_tails_and_chunk_edges(dtype, path):
    wl = _ragged_workload(SIZES, dtype)
    _report(f"ragged {dtype} path {path}, bf16 state, same state every step",
            H.run_bf16_state(wl, 8, teacher_forced=True, flags=path))
    _report(f"ragged {dtype} path {path}, bf16 state, free running", H.run_bf16_state(wl, 8, flags=path))


@pytest.mark.parametrize("name,over", [
    ("llama2_7b", dict(n_layer=2, d=256, ffn=688, vocab=1000)),
    ("llama32_1b", dict(n_layer=2, d=128, ffn=512, vocab=2000, kv_dim=32)),
    ("gpt2_small", dict(n_layer=2, d=96, vocab=1031, n_pos=64)),
    ("many_small", dict(n_tensors=300, lo=8, hi=40000)),
])
def test_small_layouts_all_elements(name, over):
    wl = workloads.build(name, **over)
    _report(f"{name} (small), bf16 state, same state every step", H.run_bf16_state(wl, 12, teacher_forced=True))
    _report(f"{name} (small), bf16 state, free running", H.run_bf16_state(wl, min(wl.n_steps, 25)))


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK], ids=["registers", "bulk"])
@pytest.mark.parametrize("optimizer", ["lion", "sgdm"])
def test_lion_and_momentum_sgd_all_elements(optimizer, path):
    for dtype in ("f32", "bf16"):
        wl = _ragged_workload(SIZES, dtype)
        _report(f"{optimizer} {dtype} path {path}, bf16 momentum, same state every step",
                H.run_bf16_state(wl, 8, optimizer=optimizer, teacher_forced=True, flags=path))
        if optimizer == "lion":       # momentum SGD's m depends on theta, so only the mode above compares it bit for bit
            _report(f"{optimizer} {dtype} path {path}, bf16 momentum, free running",
                    H.run_bf16_state(wl, 8, optimizer=optimizer, flags=path))


def test_more_partial_chunks_than_a_block_lists():
    """45 000 tensors, so that every block of the bulk-async update kernel owns about 300 partial chunks: more than it
    lists for its shared-memory ring.  One tensor in 40 is long enough to go through the ring (with a ragged tail that
    does not); those among a block's later entries take the register path like the short ones.  Both rounding modes."""
    sizes = [4100 + (i % 13) if i % 40 == 0 else 8 + (i % 29) for i in range(45000)]
    sizes[7] = 16383           # a listed chunk of two tiles
    sizes[11] = 3 * 16384 + 12000
    wl = _ragged_workload(sizes, "f32")
    _report("45000 tensors, bf16 state, same state every step",
            H.run_bf16_state(wl, 3, teacher_forced=True, flags=binding.UPDATE_PATH_BULK))
    _report("45000 tensors, bf16 state, free running", H.run_bf16_state(wl, 3, flags=binding.UPDATE_PATH_BULK))
    _report("45000 tensors, bf16 state, stochastic rounding",
            H.run_bf16_state(wl, 3, flags=binding.UPDATE_PATH_BULK, stochastic_seed=SEED))


def test_gpt2_small_all_elements():
    """Config 2 at full size (124 M parameters), every element, 20 free-running steps across the warm-up switch."""
    wl = workloads.build("gpt2_small")
    rep = H.run_bf16_state(wl, 20)
    _report("gpt2_small, bf16 state", rep)
    assert rep.clipped > 0


def test_many_small_all_elements():
    """Config 4 at full size (20 000 tensors, fp32 gradients), every element, from identical state every step."""
    wl = workloads.build("many_small")
    rep = H.run_bf16_state(wl, 8, teacher_forced=True, hyper_over=dict(lambda_abs=1e4))
    _report("many_small, bf16 state", rep)


def test_llama2_7b_sampled():
    """Config 3 at full size: all decisions, sampled elements of theta, m, v (given h_i an element's update depends on
    that element alone)."""
    wl = workloads.build("llama2_7b")
    free, _ = torch.cuda.mem_get_info()
    if free < wl.arena_elems * 10 + (8 << 30):
        pytest.skip("not enough free device memory for the 7B-shaped layout with bfloat16 state")
    rep = H.run_sampled_bf16_state(wl, 8)
    _report("llama2_7b sampled, bf16 state", rep)


# ------------------------------------------------------------------ stochastic rounding of the stored moments


@pytest.mark.parametrize("path", [binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK, binding.FUSED_SMALL],
                         ids=["registers", "bulk", "one_kernel"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_stochastic_rounding_all_elements(dtype, path):
    """adagc_set_state_rounding(STOCHASTIC): the stored moments are bit-identical to the oracle's, which draws the same
    random numbers from its own Philox4x32-10 -- through full tiles, partial chunks and ragged tails."""
    wl = _ragged_workload(SIZES, dtype)
    for forced in (True, False):
        _report(f"stochastic rounding {dtype} path {path} forced={forced}",
                H.run_bf16_state(wl, 6, teacher_forced=forced, flags=path, stochastic_seed=SEED))
    if path != binding.FUSED_SMALL:
        for optimizer in ("lion", "sgdm"):
            _report(f"stochastic rounding {optimizer} {dtype} path {path}",
                    H.run_bf16_state(wl, 5, optimizer=optimizer, teacher_forced=True, flags=path, stochastic_seed=SEED + 1))


def test_stochastic_rounding_larger_layouts_and_reproducibility():
    wl = workloads.build("gpt2_small", n_layer=2, d=384, vocab=8000, n_pos=128)
    _report("stochastic rounding, GPT-2-shaped (small)", H.run_bf16_state(wl, 12, stochastic_seed=SEED))
    wl = workloads.build("many_small", n_tensors=2000, lo=8, hi=40000)
    _report("stochastic rounding, 2000 small tensors", H.run_bf16_state(wl, 6, stochastic_seed=7, hyper_over=dict(lambda_abs=1e4)))
    # same seed: same bits; another seed: other roundings; rounding mode of an fp32-state context cannot be changed
    wl = _ragged_workload([5, 4096, 50001], "bf16")
    hp = H.hyper_of(wl)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    args = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    outs = []
    for seed in (11, 11, 12):
        opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], state_dtype=torch.bfloat16)
        opt.set_state_rounding(True, seed)
        theta, m, v, ema = _arenas(wl)
        for t in range(1, 5):
            opt.step(theta, workloads.grads_for_step(wl, t, "cuda"), m, v, ema, t, *args)
        with pytest.raises(binding.AdagcError):
            opt.step_capturable(theta, workloads.grads_for_step(wl, 5, "cuda"), m, v, ema, *args)
        outs.append((m.view(torch.int16).clone(), v.view(torch.int16).clone()))
        opt.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert (outs[0][0] != outs[2][0]).float().mean() > 0.1
    plain = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"])
    with pytest.raises(binding.AdagcError) as e:
        plain.set_state_rounding(True, 1)
    assert e.value.status == -5
    plain.close()


def test_llama2_7b_sampled_stochastic():
    wl = workloads.build("llama2_7b")
    free, _ = torch.cuda.mem_get_info()
    if free < wl.arena_elems * 10 + (8 << 30):
        pytest.skip("not enough free device memory for the 7B-shaped layout with bfloat16 state")
    _report("llama2_7b sampled, bf16 state, stochastic rounding", H.run_sampled_bf16_state(wl, 4, stochastic_seed=SEED))


def test_llama32_1b_sampled_both_rounding_modes():
    """Config 5 at full size (heavy-tailed gradients, 5 % of the tensors spiked every step, warm-up of 10 steps with
    global-norm clipping): all decisions, sampled elements of theta and of the bfloat16 m, v."""
    wl = workloads.build("llama32_1b")
    _report("llama32_1b sampled, bf16 state", H.run_sampled_bf16_state(wl, 30))
    _report("llama32_1b sampled, bf16 state, stochastic rounding", H.run_sampled_bf16_state(wl, 14, stochastic_seed=SEED))


def _arenas(wl, dev="cuda"):
    theta = workloads.init_params(wl, dev)
    m = torch.zeros(wl.arena_elems, dtype=torch.bfloat16, device=dev)
    return theta, m, torch.zeros_like(m), torch.zeros(wl.n_tensors, dtype=torch.float32, device=dev)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_other_entry_points_agree_with_adagc_step_bit_for_bit(dtype):
    """adagc_step with bfloat16 state is checked against the oracle above; the other entry points that take m and v
    (the one-kernel step, the capturable step, the host-fed step, the step that also emits bf16 parameters, the
    pre-summed step of the sharded path) must produce the same bits as adagc_step.  With fp32 gradients the step that
    emits bf16 parameters is the instantiation with the largest shared-memory ring (224 KB of the 227 KB a block may
    have)."""
    wl = _ragged_workload([5, 4096, 16384, 50001, 3 * 16384 + 9], dtype)
    hp = H.hyper_of(wl)
    offs, nums = [t.offset for t in wl.tensors], [t.numel for t in wl.tensors]
    args = (hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["wd"], hp["lambda_rel"], hp["beta"], hp["warmup"])
    n_steps = 6

    def run(kind):
        flags = binding.FUSED_SMALL if kind == "fused_small" else 0
        opt = binding.AdaGC(nums, offs, wl.torch_grad_dtype, hp["lambda_abs"], flags=flags, state_dtype=torch.bfloat16)
        theta, m, v, ema = _arenas(wl)
        lowp = torch.zeros(wl.arena_elems, dtype=torch.bfloat16, device="cuda")
        sumsq = torch.zeros(wl.n_tensors, dtype=torch.float64, device="cuda")
        for t in range(1, n_steps + 1):
            g = workloads.grads_for_step(wl, t, "cuda")
            if kind in ("step", "fused_small"):
                opt.step(theta, g, m, v, ema, t, *args)
            elif kind == "capturable":
                opt.step_capturable(theta, g, m, v, ema, *args)
            elif kind == "emit_bf16":
                opt.step_emit_bf16(theta, lowp, g, m, v, ema, t, *args)
            elif kind == "host":
                gh = g.cpu().pin_memory()
                opt.step_host(theta, torch.empty_like(g), m, v, ema, gh, t, *args)
            else:
                opt.shard_sumsq(g, sumsq)
                opt.step_presummed(theta, g, m, v, ema, sumsq, t, *args)
        st = opt.get_stats()
        assert st["status"] == 0 and st["steps_done"] == n_steps
        if kind == "emit_bf16":
            assert torch.equal(lowp, theta.to(torch.bfloat16))
        opt.close()
        return theta, m, v, ema

    want = run("step")
    for kind in ("fused_small", "capturable", "emit_bf16", "host", "presummed"):
        got = run(kind)
        for name, a, b in zip(("theta", "m", "v", "gamma"), got, want):
            if kind == "capturable" and name == "theta":      # device-side pow may round a bias correction differently
                torch.testing.assert_close(a, b, rtol=1e-6, atol=1e-9)
            else:
                assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a,
                                   b.view(torch.int16) if b.dtype == torch.bfloat16 else b), f"{kind}: {name} differs"


def test_descriptor_rules_for_bf16_state():
    """Tensor offsets must be multiples of 8 elements (the bfloat16 arenas stay 16-byte aligned), whatever the
    gradient dtype; an fp32 arena passed where the context expects bfloat16 is the caller's error, caught in the binding."""
    with pytest.raises(binding.AdagcError) as e:
        binding.AdaGC([4, 8], [0, 4], torch.float32, state_dtype=torch.bfloat16)
    assert e.value.status == -2
    opt = binding.AdaGC([4, 8], [0, 8], torch.float32, state_dtype=torch.bfloat16)
    theta = torch.zeros(16, device="cuda")
    with pytest.raises(AssertionError):
        opt.step(theta, theta, theta, theta, torch.zeros(2, device="cuda"), 1, 1e-3, 0.9, 0.95, 1e-8, 0.1, 1.04, 0.99, 0)
    opt.close()
