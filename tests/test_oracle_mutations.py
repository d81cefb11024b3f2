"""Are the pins sharp?  Plant one plausible mistake at a time in a copy of the numpy oracle (on the
CPU, never in the CUDA path) and require that at least one pin of test_oracle_pins.py fails."""
import importlib.util
import os
import sys
import types

import numpy as np
import pytest

import test_oracle_pins as pins
import test_oracle_pins_bf16_state as pins_bf

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "adagc_oracle.py")

MUTATIONS = {
    "raw norm enters the EMA": ("c[i] = thr  ", "c[i] = n[i]  "),
    "non-strict comparison": ("if n[i] > thr:", "if n[i] >= thr:"),
    "warm-up seeds gamma with the raw norm": ("c[i] = h_t * n[i]", "c[i] = n[i]"),
    "warm-up keeps the maximum": ("else min(gam[i], c[i])", "else max(gam[i], c[i])"),
    "second moment of the unclipped gradient": ("(1.0 - hp.beta2) * gh * gh",
                                                "(1.0 - hp.beta2) * np.asarray(g, dtype=np.float64) ** 2"),
    "no bias correction of m": ("m_hat = m1 / (1.0 - hp.beta1 ** step)", "m_hat = m1"),
    "bias correction of v with beta1": ("v_hat = v1 / (1.0 - hp.beta2 ** step)", "v_hat = v1 / (1.0 - hp.beta1 ** step)"),
    "weight decay with the wrong sign": ("th - hp.lr * hp.wd * th", "th + hp.lr * hp.wd * th"),
    "warm-up one step short": ("if step <= hp.warmup:", "if step < hp.warmup:"),
    "lambda_rel dropped from the threshold": ("thr = hp.lambda_rel * gam[i]", "thr = gam[i]"),
    "epsilon inside the square root": ("(np.sqrt(v_hat) + hp.eps)", "np.sqrt(v_hat + hp.eps)"),
    "clip factor inverted": ("h[i] = thr / n[i]", "h[i] = n[i] / thr"),
    "global threshold uses lambda_rel": ("h_t = hp.lambda_abs / G if clip_all", "h_t = hp.lambda_rel / G if clip_all"),
    "EMA weights swapped": ("gam[i] = hp.beta * gam[i] + (1.0 - hp.beta) * c[i]",
                            "gam[i] = (1.0 - hp.beta) * gam[i] + hp.beta * c[i]"),
    "first moment of the unclipped gradient": ("(1.0 - hp.beta1) * gh", "(1.0 - hp.beta1) * np.asarray(g, dtype=np.float64)"),
    "sum instead of sum of squares": ("float(np.sum(x * x))", "float(np.sum(np.abs(x)))"),
}

PINS = [pins.test_norm_matches_fsum_and_linalg, pins.test_norm_closed_forms, pins.test_hand_worked_example,
        pins.test_clipped_run_matches_library_adamw_on_library_clipped_grads, pins.test_first_step_closed_form,
        pins.test_lemma1_invariant, pins.test_spike_is_scaled_to_lambda_rel_gamma,
        pins.test_scale_equivariance_power_of_two, pins.test_warmup_switch_and_min_seeding,
        pins.test_degenerate_norms]


def _mutant(old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation anchor {old!r} must occur exactly once in the oracle"
    mod = types.ModuleType("adagc_oracle_mutant")
    mod.__file__ = SRC
    sys.modules[mod.__name__] = mod                      # dataclasses look the module up by name
    exec(compile(text.replace(old, new), SRC, "exec"), mod.__dict__)

    class Impl:
        name = "mutant"

        @staticmethod
        def sumsq(g):
            return mod.sumsq(g)

        @staticmethod
        def decisions(s, gamma, step, hp):
            r = mod.clip_decisions(s, gamma, step, mod.Hyper(**hp.__dict__), np.float32)
            return dict(norm=r.norm, h=r.h, flag=r.flag, clipped=r.clipped, gamma=r.gamma,
                        global_norm=r.global_norm, margin=r.margin)

        @staticmethod
        def adamw(theta, g, m, v, h, step, hp):
            return mod.adamw_update(theta, g, m, v, h, step, mod.Hyper(**hp.__dict__), np.float32)

    return Impl


def test_unmutated_copy_passes_every_pin():
    impl = _mutant("sum_j g_j^2 of one tensor", "sum_j g_j^2 of one tensor")
    for pin in PINS:
        pin(impl)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_every_planted_mistake_is_caught(name):
    impl = _mutant(*MUTATIONS[name])
    caught = []
    for pin in PINS:
        try:
            pin(impl)
        except AssertionError:
            caught.append(pin.__name__)
        except Exception as e:                            # a mistake may also crash a pin; that counts
            caught.append(f"{pin.__name__} ({type(e).__name__})")
    assert caught, f"no pin notices: {name}"


# ---------------------------------------------------------------- the optimizer variants and the Section 5 ablations
VARIANT_MUTATIONS = {
    "Lion: momentum interpolation with beta2": ("a, b = beta1 * mm, (1.0 - beta1) * gh", "a, b = beta2 * mm, (1.0 - beta2) * gh"),
    "Lion: sign of the step flipped": ("th1 = th - lr * (np.sign(c) + wd * th)", "th1 = th + lr * (np.sign(c) + wd * th)"),
    "Lion: stored momentum uses beta1": ("m1 = beta2 * mm + (1.0 - beta2) * gh", "m1 = beta1 * mm + (1.0 - beta1) * gh"),
    "Lion: unclipped gradient": ("gh = float(h) * np.asarray(g, dtype=np.float64)\n    a, b", "gh = np.asarray(g, dtype=np.float64)\n    a, b"),
    "SGD: decay with the wrong sign": ("+ wd * th\n    m1 = momentum", "- wd * th\n    m1 = momentum"),
    "SGD: dampened momentum": ("m1 = momentum * np.asarray(m, dtype=np.float64) + d", "m1 = momentum * np.asarray(m, dtype=np.float64) + (1.0 - momentum) * d"),
    "thresholded init keeps the larger value": ("gam[i] = c[i] if c[i] < ema_cap else ema_cap", "gam[i] = c[i] if c[i] > ema_cap else ema_cap"),
    "thresholded init keeps a running minimum": ("gam[i] = c[i] if c[i] < ema_cap else ema_cap", "gam[i] = min(gam[i], c[i], ema_cap)"),
    "thresholded init not applied to the seed of T_start = 0": ("if ema_cap is not None and ema_cap > 0 and not gam[i] < ema_cap:", "if False:"),
    "constant init is overwritten at t = 1": ("seed = step == 1 and not keep_initial", "seed = step == 1"),
    "Global AdaGC uses the largest tensor only": ("one = clip_decisions([float(np.sum(s_all))]", "one = clip_decisions([float(np.max(s_all))]"),
    "Global AdaGC keeps per-tensor gamma": ("np.full(T, one.gamma[0], dtype=state_dtype), one.global_norm", "np.asarray(gamma_prev, dtype=state_dtype), one.global_norm"),
}

VARIANT_PINS = [(pins.test_lion_closed_forms, ("numpy",)), (pins.test_lion_brute_force_and_oracles_agree, ()),
                (pins.test_sgdm_matches_library_sgd, ("numpy",)),
                (pins.test_thresholded_initialization_hand_values_and_special_cases, ("numpy",)),
                (pins.test_thresholded_initialization_brute_force_and_oracles_agree, ()),
                (pins.test_keep_initial_uses_the_callers_gamma_from_the_first_step, ("numpy",)),
                (pins.test_global_adaptive_is_the_algorithm_on_the_concatenated_gradient, ("numpy",))]


def _mutant_module(old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation anchor {old!r} must occur exactly once in the oracle"
    mod = types.ModuleType("adagc_oracle_variant_mutant")
    mod.__file__ = SRC
    sys.modules[mod.__name__] = mod
    exec(compile(text.replace(old, new), SRC, "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(VARIANT_MUTATIONS))
def test_every_planted_mistake_in_a_variant_is_caught(name, monkeypatch):
    """The same game for Lion, momentum SGD and the ablation variants: the pins call the numpy oracle through the
    name `npo` of their module, which is pointed at a mutated copy for the duration of the test."""
    monkeypatch.setattr(pins, "npo", _mutant_module(*VARIANT_MUTATIONS[name]))
    caught = []
    for pin, args in VARIANT_PINS:
        try:
            pin(*args)
        except AssertionError:
            caught.append(pin.__name__)
        except Exception as e:
            caught.append(f"{pin.__name__} ({type(e).__name__})")
    assert caught, f"no pin notices: {name}"


def test_unmutated_variant_pins_pass():
    for pin, args in VARIANT_PINS:
        pin(*args)


# ---------------------------------------------------------------- optimizer state stored as bfloat16
BF16_STATE_MUTATIONS = {
    "moments truncated instead of rounded": ("np.ldexp(np.rint(q), p - 7)", "np.ldexp(np.trunc(q), p - 7)"),
    "ties rounded away from zero": ("np.ldexp(np.rint(q), p - 7)", "np.ldexp(np.sign(q) * np.floor(np.abs(q) + 0.5), p - 7)"),
    "subnormals rounded on the grid of normal numbers": ("p = np.maximum(e - 1, -126) ", "p = e - 1 "),
    "v stored unrounded": ("round_to_bf16(v1).astype(np.float32))", "v1.astype(np.float32))"),
    "m stored unrounded": ("round_to_bf16(m1).astype(np.float32), round_to_bf16(v1)", "m1.astype(np.float32), round_to_bf16(v1)"),
    "theta updated from the rounded first moment": ("m_hat = m1 / (1.0 - hp.beta1 ** step)",
                                                    "m_hat = (m1 if moment_dtype is None else round_to_bf16(m1)) / (1.0 - hp.beta1 ** step)"),
    "theta updated from the rounded second moment": ("v_hat = v1 / (1.0 - hp.beta2 ** step)",
                                                     "v_hat = (v1 if moment_dtype is None else round_to_bf16(v1)) / (1.0 - hp.beta2 ** step)"),
    "Lion momentum stored unrounded": ("m1.astype(state_dtype) if moment_dtype is None else round_to_bf16(m1).astype(np.float32))\n    if return_margin:",
                                       "m1.astype(state_dtype))\n    if return_margin:"),
    "SGD: theta sees the rounded momentum": ("th1 = th - lr * m1 ", "th1 = th - lr * (m1 if moment_dtype is None else round_to_bf16(m1)) "),
    "SGD momentum stored unrounded": ("return th1.astype(state_dtype), m1.astype(state_dtype) if moment_dtype is None else round_to_bf16(m1).astype(np.float32)",
                                      "return th1.astype(state_dtype), m1.astype(state_dtype)"),
    "flip distance ignores the denser values below a power of two": ("dist = np.where(low_edge, np.minimum(dist, frac + 0.25), dist)",
                                                                     "dist = dist + 0.0 * low_edge"),
}

BF16_STATE_MUTATIONS.update({
    "Philox: key not bumped between rounds": ("        if r < 9:\n            k0, k1 = (k0 + np.uint64(PHILOX_W0)) & mask, (k1 + np.uint64(PHILOX_W1)) & mask",
                                              "        if False:\n            pass"),
    "Philox: nine rounds": ("    for r in range(10):\n        p0, p1 = np.uint64(PHILOX_M0)", "    for r in range(9):\n        p0, p1 = np.uint64(PHILOX_M0)"),
    "Philox: multipliers swapped": ("p0, p1 = np.uint64(PHILOX_M0) * c0, np.uint64(PHILOX_M1) * c2", "p0, p1 = np.uint64(PHILOX_M1) * c0, np.uint64(PHILOX_M0) * c2"),
    "stochastic rounding: m and v use the same half of the word": ("(word >> np.uint32(16)).astype(np.uint32)", "(word & np.uint32(0xFFFF)).astype(np.uint32)"),
    "stochastic rounding: one generator call per element instead of per four": ("q = index >> np.uint64(2)", "q = index"),
    "stochastic rounding: step not in the counter": ("np.full(q.shape, step & 0xFFFFFFFF, np.uint64)", "np.full(q.shape, 0, np.uint64)"),
    "stochastic rounding: always toward zero": ("out = (((u + np.asarray(r16, np.uint64)) >> np.uint64(16))", "out = (((u + 0 * np.asarray(r16, np.uint64)) >> np.uint64(16))"),
    "stochastic rounding: random number twice as large": ("out = (((u + np.asarray(r16, np.uint64)) >> np.uint64(16))", "out = (((u + 2 * np.asarray(r16, np.uint64)) >> np.uint64(16))"),
})

BF16_STATE_PINS = [(pins_bf.test_rounding_matches_the_library_conversion_and_ties_go_to_even, ()),
                   (pins_bf.test_rounding_margin_is_the_distance_to_a_flip, ()),
                   (pins_bf.test_one_step_from_a_given_state_matches_library_adamw, (pins_bf.NumpyBF, 7)),
                   (pins_bf.test_theta_is_the_fp32_state_paths_theta_bit_for_bit, (pins_bf.NumpyBF,)),
                   (pins_bf.test_lion_and_sgdm_store_the_nearest_bf16_and_leave_theta_alone, ("numpy",)),
                   (pins_bf.test_c_oracle_counts_decisions_close_to_a_flip, ()),
                   (pins_bf.test_philox_known_answers, ()),
                   (pins_bf.test_stochastic_rounding_is_exactly_unbiased_and_leaves_bf16_values_alone, ()),
                   (pins_bf.test_stochastic_step_is_the_nearest_rounding_steps_value_rounded_with_the_stated_random_numbers, ())]


@pytest.mark.parametrize("name", sorted(BF16_STATE_MUTATIONS))
def test_every_planted_mistake_in_the_bf16_state_is_caught(name, monkeypatch):
    monkeypatch.setattr(pins_bf, "npo", _mutant_module(*BF16_STATE_MUTATIONS[name]))
    caught = []
    for pin, args in BF16_STATE_PINS:
        try:
            pin(*args)
        except AssertionError:
            caught.append(pin.__name__)
        except Exception as e:
            caught.append(f"{pin.__name__} ({type(e).__name__})")
    assert caught, f"no pin notices: {name}"


def test_unmutated_bf16_state_pins_pass():
    for pin, args in BF16_STATE_PINS:
        pin(*args)
