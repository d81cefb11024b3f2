"""Are the pins sharp?  Plant one plausible mistake at a time in a copy of the numpy oracle (on the
CPU, never in the CUDA path) and require that at least one pin of test_oracle_pins.py fails."""
import importlib.util
import os
import sys
import types

import numpy as np
import pytest

import test_oracle_pins as pins

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
