"""Pins for the CPU oracles (numpy and C) against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each pin is something other than the oracle's
own formula: a closed form, an invariant (Lemma 1), a special case that reduces to a library
routine (torch.optim.AdamW, torch.nn.utils.clip_grad_norm_, math.fsum, numpy.linalg.norm),
the hand-worked example under tests/golden/, or a brute-force scalar loop.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import adagc_oracle as npo
from oracle import c_oracle as co

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- adapters
class NumpyImpl:
    name = "numpy"

    @staticmethod
    def sumsq(g):
        return npo.sumsq(g)

    @staticmethod
    def decisions(s, gamma, step, hp):
        r = npo.clip_decisions(s, gamma, step, hp, np.float32)
        return dict(norm=r.norm, h=r.h, flag=r.flag, clipped=r.clipped, gamma=r.gamma,
                    global_norm=r.global_norm, margin=r.margin)

    @staticmethod
    def adamw(theta, g, m, v, h, step, hp):
        return npo.adamw_update(theta, g, m, v, h, step, hp, np.float32)


class CImpl:
    name = "c"

    @staticmethod
    def sumsq(g):
        return co.sumsq(np.ascontiguousarray(g, dtype=np.float32))

    @staticmethod
    def decisions(s, gamma, step, hp):
        gam = np.array(gamma, dtype=np.float32)
        r = co.clip_decisions(np.asarray(s, np.float64), gam, step, hp.lambda_rel, hp.beta,
                              hp.lambda_abs, hp.warmup)
        return r

    @staticmethod
    def adamw(theta, g, m, v, h, step, hp):
        th, mm, vv = (np.array(a, dtype=np.float32) for a in (theta, m, v))
        co.adamw_update(th, np.ascontiguousarray(g, dtype=np.float32), mm, vv, h, step,
                        hp.lr, hp.beta1, hp.beta2, hp.eps, hp.wd)
        return th, mm, vv


IMPLS = [NumpyImpl, CImpl]


def run(impl, params, grads_per_step, hp):
    """Algorithm 1 over a list of tensors with fp32 storage; returns per-step decisions + state."""
    theta = [np.array(p, dtype=np.float32) for p in params]
    m = [np.zeros_like(p) for p in theta]
    v = [np.zeros_like(p) for p in theta]
    gamma = np.zeros(len(theta), dtype=np.float32)
    hist = []
    for t, grads in enumerate(grads_per_step, start=1):
        s = [impl.sumsq(g) for g in grads]
        r = impl.decisions(s, gamma, t, hp)
        gamma = np.array(r["gamma"], dtype=np.float32)
        for i, g in enumerate(grads):
            theta[i], m[i], v[i] = impl.adamw(theta[i], g, m[i], v[i], float(r["h"][i]), t, hp)
        hist.append({k: np.array(val, copy=True) for k, val in r.items()})
    return hist, theta, m, v, gamma


def f32_exact(x):
    """Random values that are exactly representable in fp32 (so both oracles see the same bits)."""
    return np.asarray(x, dtype=np.float32)


# ----------------------------------------------------------------------------- a1: the norm
@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_norm_matches_fsum_and_linalg(impl):
    rng = np.random.RandomState(1)
    for n in (1, 2, 3, 7, 64, 1000, 4097, 100003):
        g = f32_exact(rng.standard_t(2, size=n) * 1e-3)
        exact = math.fsum(float(x) * float(x) for x in g)
        assert impl.sumsq(g) == pytest.approx(exact, rel=1e-15)
        assert math.sqrt(impl.sumsq(g)) == pytest.approx(np.linalg.norm(g.astype(np.float64)), rel=1e-14)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_norm_closed_forms(impl):
    assert math.sqrt(impl.sumsq(f32_exact([3, 4]))) == 5.0
    assert math.sqrt(impl.sumsq(f32_exact([5, 0, 12, 0]))) == 13.0
    for c, n in ((0.5, 4096), (2.0, 65536), (0.25, 10 ** 6)):
        assert math.sqrt(impl.sumsq(np.full(n, c, np.float32))) == pytest.approx(c * math.sqrt(n), rel=1e-15)
    assert impl.sumsq(np.zeros(17, np.float32)) == 0.0


def test_c_oracle_bf16_inputs_and_rounding():
    rng = np.random.RandomState(2)
    x = torch.from_numpy(rng.standard_t(3, size=20001).astype(np.float32) * 1e-4)
    xb = x.to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16)
    exact = math.fsum(float(v) ** 2 for v in xb.double().numpy())
    assert co.sumsq(bits) == pytest.approx(exact, rel=1e-15)
    # double -> bf16 rounding of the C oracle vs the library's round-to-nearest-even conversion
    vals = np.concatenate([x.numpy().astype(np.float64), [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38,
                                                           1e-40, -1e-39, 2.0 ** -133, 65280.0, 3.3961775e38]])
    vals = vals.astype(np.float32).astype(np.float64)        # both sides see the same fp32-representable values
    want = torch.from_numpy(vals.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([co.double_to_bf16_bits(v) for v in vals], dtype=np.uint16)
    np.testing.assert_array_equal(got, want)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert co.double_to_bf16_bits(1.0 + 2.0 ** -8) == 0x3F80
    assert co.double_to_bf16_bits(1.0 + 3 * 2.0 ** -8) == 0x3F82


# ----------------------------------------------------------------------------- hand-worked example
def test_golden_fixture_equals_its_exact_derivation():
    """The stored hand-worked table is reproduced by exact rational arithmetic (no oracle involved)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_worked_example", os.path.join(GOLDEN, "make_worked_example.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    for r, s in zip(mod.derive(), _golden()["steps"]):
        assert r["norm"] == s["norm"] and r["h"] == s["h"] and r["flag"] == s["flag"] and r["gamma"] == s["gamma"]
        if "global_norm" in s:
            assert r["global_norm_sq"] == s["global_norm"] ** 2
        if "global_norm_sq" in s:
            assert r["global_norm_sq"] == s["global_norm_sq"]


def _golden():
    with open(os.path.join(GOLDEN, "worked_example.json")) as f:
        return json.load(f)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_hand_worked_example(impl):
    gold = _golden()
    hp = npo.Hyper(**gold["hyper"])
    params = [gold["theta0"]["A"], gold["theta0"]["B"]]
    grads = [[f32_exact(s["gA"]), f32_exact(s["gB"])] for s in gold["steps"]]
    hist, theta, m, v, gamma = run(impl, params, grads, hp)
    for s, r in zip(gold["steps"], hist):
        np.testing.assert_array_equal(r["norm"], s["norm"])
        np.testing.assert_array_equal(r["h"], s["h"])
        np.testing.assert_array_equal(np.asarray(r["flag"], dtype=int), s["flag"])
        np.testing.assert_array_equal(np.asarray(r["gamma"], dtype=np.float64), s["gamma"])
        if "global_norm" in s:
            assert float(r["global_norm"]) == s["global_norm"]
        if "global_norm_sq" in s:
            assert float(r["global_norm"]) == pytest.approx(math.sqrt(s["global_norm_sq"]), rel=1e-15)
    # clipped norm equals lambda_rel * gamma_{t-1} exactly when the clip is active (Section 4.2)
    assert hist[2]["clipped"][0] == 1.5 * 1.25 and hist[3]["clipped"][0] == 1.5 * 1.5625
    # theta after the whole run: the library AdamW fed with the hand-derived clip factors
    want = _torch_adamw([np.array(p, np.float64) for p in params],
                        [[np.asarray(g, np.float64) * h for g, h in zip(gs, s["h"])]
                         for gs, s in zip(grads, gold["steps"])], hp)
    for a, b in zip(theta, want):
        np.testing.assert_allclose(a, b, rtol=3e-7, atol=0)   # fp32 storage vs float64 library run


def test_second_hand_worked_example_with_printed_parameters():
    """The decimal variant of the example (g_A = (0.6, 0.8) at t = 2), whose parameters are printed to 10 digits after
    every step: the float64-state oracle reproduces the table to rounding and every printed theta to 1e-9; the fixture
    itself is re-derived in 50-digit decimal arithmetic by tests/golden/make_worked_example.py, without the oracle.
    (The first fixture uses (0.75, 1) instead, so that every input is exact in binary and the fp32 paths -- the C oracle
    and the GPU -- can be required to reproduce its table bit for bit.)"""
    with open(os.path.join(GOLDEN, "worked_example_decimal.json")) as f:
        gold = json.load(f)
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_worked_example", os.path.join(GOLDEN, "make_worked_example.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    derived = mod.derive_theta(mod.GRADS_DECIMAL, [gold["theta0"]["A"], gold["theta0"]["B"]])
    hp = npo.Hyper(**gold["hyper"])
    ref = npo.AdaGCAdamW([np.array(gold["theta0"]["A"]), np.array(gold["theta0"]["B"])], hp, np.float64)
    for s, d in zip(gold["steps"], derived):
        r = ref.step([np.array(s["gA"], np.float64), np.array(s["gB"], np.float64)])
        np.testing.assert_allclose(r.norm, s["norm"], rtol=1e-15, atol=0)
        np.testing.assert_allclose(r.h, s["h"], rtol=1e-15)
        np.testing.assert_array_equal(r.flag.astype(int), s["flag"])
        np.testing.assert_allclose(r.gamma, s["gamma"], rtol=1e-15)
        for got, printed, exact in zip(ref.theta, (s["theta_A"], s["theta_B"]), d):
            np.testing.assert_allclose(got, printed, rtol=0, atol=1e-9)        # the printed 10 digits
            np.testing.assert_allclose(got, exact, rtol=1e-13, atol=0)         # the 50-digit derivation
    # the C oracle (fp32 storage) on the same inputs rounded to fp32
    theta = [np.array(gold["theta0"]["A"], np.float32), np.array(gold["theta0"]["B"], np.float32)]
    grads = [[f32_exact(s["gA"]), f32_exact(s["gB"])] for s in gold["steps"]]
    hist, th, _, _, _ = run(CImpl, theta, grads, hp)
    for s, r in zip(gold["steps"], hist):
        np.testing.assert_array_equal(np.asarray(r["flag"], int), s["flag"])
        np.testing.assert_allclose(r["h"], s["h"], rtol=1e-7)
    np.testing.assert_allclose(np.concatenate(th), gold["steps"][-1]["theta_A"] + gold["steps"][-1]["theta_B"], rtol=5e-7)


def _torch_adamw(params, clipped_grads_per_step, hp, dtype=torch.float64):
    ps = [torch.tensor(p, dtype=dtype, requires_grad=True) for p in params]
    opt = torch.optim.AdamW(ps, lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps,
                            weight_decay=hp.wd, foreach=False)
    for grads in clipped_grads_per_step:
        for p, g in zip(ps, grads):
            p.grad = torch.tensor(np.asarray(g), dtype=dtype)
        opt.step()
    return [p.detach().numpy() for p in ps]


# ----------------------------------------------------------------------------- a6/a7: AdamW
def test_all_unclipped_is_plain_adamw_float64():
    """With every h = 1 Algorithm 1 is AdamW: compare the float64-state oracle with torch.optim.AdamW."""
    rng = np.random.RandomState(3)
    shapes = [(5, 7), (11,), (3, 4, 2)]
    params = [rng.normal(0, 0.02, size=s) for s in shapes]
    base = [rng.normal(0, 1e-3, size=s) for s in shapes]
    # shrinking norms: after seeding at step 1 nothing ever exceeds lambda_rel * gamma
    grads = [[b * (0.97 ** t) * np.sign(rng.normal(size=b.shape)) for b in base] for t in range(40)]
    for warmup in (0, 5):
        hp = npo.Hyper(lr=1e-2, warmup=warmup, lambda_abs=1e9)
        opt = npo.AdaGCAdamW(params, hp, state_dtype=np.float64)
        for gs in grads:
            r = opt.step(gs)
            assert not r.flag.any() and (r.h == 1.0).all()
        want = _torch_adamw(params, grads, hp)
        for a, b in zip(opt.theta, want):
            np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-18)
        # and bit-identical to the oracle's own clip-free AdamW loop
        th, m, v = [p.copy() for p in params], [np.zeros_like(p) for p in params], [np.zeros_like(p) for p in params]
        for t, gs in enumerate(grads, start=1):
            for i, g in enumerate(gs):
                th[i], m[i], v[i] = npo.adamw_update(th[i], g, m[i], v[i], 1.0, t, hp, np.float64)
        for a, b in zip(opt.theta, th):
            np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_clipped_run_matches_library_adamw_on_library_clipped_grads(impl):
    """Whole path vs library routines: per-tensor clip by torch's clip_grad_norm_ (its 1e-6 in the
    denominator makes this a loose check) feeding torch.optim.AdamW."""
    rng = np.random.RandomState(4)
    shapes = [(64, 3), (200,), (9, 9)]
    params = [f32_exact(rng.normal(0, 0.02, size=s)) for s in shapes]
    steps = 30
    grads = []
    for t in range(steps):
        gs = [f32_exact(rng.normal(0, 1.0, size=s)) for s in shapes]
        if t in (12, 20):
            gs[t % 3] = gs[t % 3] * np.float32(50.0)
        grads.append(gs)
    hp = npo.Hyper(lr=1e-3, warmup=4, lambda_abs=10.0, lambda_rel=1.04, beta=0.9)
    hist, theta, m, v, gamma = run(impl, params, grads, hp)
    assert any(r["flag"].any() for r in hist[4:])          # spikes were clipped
    assert all(r["flag"].all() for r in hist[:4])          # warm-up clipped globally (norm ~ 21 > 10)
    # library replay
    ps = [torch.tensor(p, dtype=torch.float64, requires_grad=True) for p in params]
    opt = torch.optim.AdamW(ps, lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps, weight_decay=hp.wd)
    gam = [None] * len(ps)
    for t, gs in enumerate(grads, start=1):
        for p, g in zip(ps, gs):
            p.grad = torch.tensor(g, dtype=torch.float64)
        if t <= hp.warmup:
            torch.nn.utils.clip_grad_norm_(ps, hp.lambda_abs)
            for i, p in enumerate(ps):
                n = float(p.grad.norm())
                gam[i] = n if t == 1 else min(gam[i], n)
        else:
            for i, p in enumerate(ps):
                torch.nn.utils.clip_grad_norm_([p], hp.lambda_rel * gam[i])
                gam[i] = hp.beta * gam[i] + (1 - hp.beta) * float(p.grad.norm())
        opt.step()
    for a, p in zip(theta, ps):
        np.testing.assert_allclose(a, p.detach().numpy(), rtol=2e-5, atol=1e-7)
    np.testing.assert_allclose(gamma, gam, rtol=1e-5)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_first_step_closed_form(impl):
    """At t = 1, m_hat = g_hat and v_hat = g_hat^2: theta_1 = theta_0 (1 - lr wd) - lr g_hat / (|g_hat| + eps)."""
    rng = np.random.RandomState(5)
    theta0 = f32_exact(rng.normal(size=257))
    g = f32_exact(rng.normal(size=257) * 1e-2)
    g[::10] = 0.0
    hp = npo.Hyper(lr=1e-2, wd=0.1, eps=1e-8)
    for h in (1.0, 0.25):
        th, m, v = impl.adamw(theta0, g, np.zeros_like(g), np.zeros_like(g), h, 1, hp)
        gh = h * g.astype(np.float64)
        want = theta0.astype(np.float64) * (1 - hp.lr * hp.wd) - hp.lr * gh / (np.abs(gh) + hp.eps)
        np.testing.assert_allclose(th, want, rtol=2e-7, atol=1e-9)
        np.testing.assert_allclose(m, (1 - hp.beta1) * gh, rtol=1e-7)
        np.testing.assert_allclose(v, (1 - hp.beta2) * gh * gh, rtol=2e-7)
        # zero-gradient elements only decay
        np.testing.assert_allclose(th[::10], theta0[::10].astype(np.float64) * (1 - hp.lr * hp.wd), rtol=1e-7)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_lemma1_invariant(impl):
    """Lemma 1: m^2 <= v / ((1 - beta1^2/beta2)(1 - beta2)) for every element and step."""
    rng = np.random.RandomState(6)
    n = 512
    hp = npo.Hyper(beta1=0.9, beta2=0.95, warmup=3, lambda_abs=0.05)
    zeta = hp.beta1 ** 2 / hp.beta2
    bound = 1.0 / ((1 - zeta) * (1 - hp.beta2))
    grads = [[f32_exact(rng.standard_t(2, size=n) * 1e-3 * (100.0 if t == 15 else 1.0))] for t in range(40)]
    theta, m, v = [f32_exact(rng.normal(size=n))], None, None
    gamma = np.zeros(1, np.float32)
    mm, vv = np.zeros(n, np.float32), np.zeros(n, np.float32)
    th = theta[0]
    for t, gs in enumerate(grads, start=1):
        r = impl.decisions([impl.sumsq(gs[0])], gamma, t, hp)
        gamma = np.array(r["gamma"], np.float32)
        th, mm, vv = impl.adamw(th, gs[0], mm, vv, float(r["h"][0]), t, hp)
        lhs, rhs = mm.astype(np.float64) ** 2, bound * vv.astype(np.float64)
        assert (lhs <= rhs * (1 + 1e-5) + 1e-40).all()


# ----------------------------------------------------------------------------- a3/a4: AdaGC branch
@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_spike_is_scaled_to_lambda_rel_gamma(impl):
    rng = np.random.RandomState(7)
    hp = npo.Hyper(warmup=0, lambda_rel=1.04, beta=0.99)
    g0 = f32_exact(rng.normal(size=1000) * 1e-3)
    gamma = np.zeros(1, np.float32)
    r = impl.decisions([impl.sumsq(g0)], gamma, 1, hp)
    assert not r["flag"][0] and r["h"][0] == 1.0
    gamma = np.array(r["gamma"], np.float32)
    assert float(gamma[0]) == pytest.approx(math.sqrt(impl.sumsq(g0)), rel=1e-7)
    # calm step: h is exactly 1
    g1 = f32_exact(g0 * np.float32(1.03))
    r1 = impl.decisions([impl.sumsq(g1)], gamma, 2, hp)
    assert not r1["flag"][0] and r1["h"][0] == 1.0 and r1["clipped"][0] == r1["norm"][0]
    # spike: the clipped gradient has norm lambda_rel * gamma_{t-1}
    g2 = f32_exact(g0 * np.float32(100.0))
    r2 = impl.decisions([impl.sumsq(g2)], gamma, 2, hp)
    assert r2["flag"][0] and r2["h"][0] < 1.0
    thr = hp.lambda_rel * float(gamma[0])
    assert r2["clipped"][0] == thr
    ghat = float(r2["h"][0]) * g2.astype(np.float64)
    assert np.linalg.norm(ghat) == pytest.approx(thr, rel=1e-12)
    # the clipped (not the raw) norm enters the EMA
    assert float(r2["gamma"][0]) == pytest.approx(hp.beta * float(gamma[0]) + (1 - hp.beta) * thr, rel=1e-7)
    raw_ema = hp.beta * float(gamma[0]) + (1 - hp.beta) * float(r2["norm"][0])     # what the raw norm would give
    assert float(r2["gamma"][0]) < 0.75 * raw_ema


def test_ema_closed_forms_long_run():
    """Scalar-only long runs in float64 state: geometric approach when never clipped, geometric
    growth (beta + (1-beta) lambda_rel)^t when always clipped."""
    hp = npo.Hyper(warmup=0, lambda_rel=1.04, beta=0.99)
    gamma = np.array([2.0])
    n = 1.5                                                    # below threshold forever
    g0 = float(gamma[0])
    for t in range(2, 2000):
        r = npo.clip_decisions([n * n], gamma, t, hp, np.float64)
        assert not r.flag[0]
        gamma = r.gamma
        assert gamma[0] == pytest.approx(n + (g0 - n) * hp.beta ** (t - 1), rel=1e-12)
    gamma = np.array([1.0])
    rate = hp.beta + (1 - hp.beta) * hp.lambda_rel           # 1.0004 at the defaults
    assert rate == pytest.approx(1.0004, rel=1e-12)
    for t in range(2, 12000):
        r = npo.clip_decisions([100.0 ** 2], gamma, t, hp, np.float64)
        gamma = r.gamma
        if gamma[0] * hp.lambda_rel < 100.0:
            assert r.flag[0]
    k = math.log(100.0 / hp.lambda_rel) / math.log(rate)       # steps until a x100 level shift is absorbed
    assert 11400 < k < 11520
    gamma = np.array([1.0])
    for t in range(2, 2 + 500):
        gamma = npo.clip_decisions([100.0 ** 2], gamma, t, hp, np.float64).gamma
    assert gamma[0] == pytest.approx(rate ** 500, rel=1e-12)


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_scale_equivariance_power_of_two(impl):
    """Scaling all gradients (and lambda_abs) by 2^k leaves flags and h bit-identical and scales gamma by 2^k."""
    rng = np.random.RandomState(8)
    shapes = [(330,), (1000,), (70, 9)]
    params = [f32_exact(rng.normal(size=s)) for s in shapes]
    grads = []
    for t in range(25):
        gs = [f32_exact(rng.normal(size=s) * 1e-2) for s in shapes]
        if t in (2, 9, 15, 21):
            gs[t % 3] = gs[t % 3] * np.float32(64.0)
        grads.append(gs)
    hp = npo.Hyper(warmup=4, lambda_abs=0.5)
    h1, *_, gam1 = run(impl, params, grads, hp)
    for k in (-6, 5):
        c = np.float32(2.0 ** k)
        hp2 = npo.Hyper(warmup=4, lambda_abs=0.5 * float(c))
        h2, *_, gam2 = run(impl, params, [[g * c for g in gs] for gs in grads], hp2)
        for a, b in zip(h1, h2):
            np.testing.assert_array_equal(a["flag"], b["flag"])
            np.testing.assert_array_equal(a["h"], b["h"])
            np.testing.assert_array_equal(np.asarray(a["gamma"], np.float64) * float(c), np.asarray(b["gamma"], np.float64))
    steady = np.array([a["flag"] for a in h1[4:]])
    assert steady.any() and not steady.all()
    assert h1[2]["flag"].all() and not h1[1]["flag"].any()       # warm-up clipped once, globally
    assert h1[2]["flag"].all() and not h1[1]["flag"].any()       # warm-up clipped once, globally


def test_scale_equivariance_general_factor_float64():
    rng = np.random.RandomState(9)
    params = [rng.normal(size=50), rng.normal(size=8)]
    grads = [[rng.standard_t(3, size=50) * (30 if t == 9 else 1), rng.normal(size=8)] for t in range(20)]
    hp = npo.Hyper(warmup=3, lambda_abs=2.0)
    a = npo.AdaGCAdamW(params, hp, np.float64)
    c = 0.37
    b = npo.AdaGCAdamW(params, npo.Hyper(warmup=3, lambda_abs=2.0 * c), np.float64)
    for gs in grads:
        ra, rb = a.step(gs), b.step([g * c for g in gs])
        np.testing.assert_array_equal(ra.flag, rb.flag)
        np.testing.assert_allclose(ra.h, rb.h, rtol=1e-12)
        np.testing.assert_allclose(ra.gamma * c, rb.gamma, rtol=1e-12)


# ----------------------------------------------------------------------------- a2/a4: warm-up
@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_warmup_switch_and_min_seeding(impl):
    rng = np.random.RandomState(10)
    shapes = [(40,), (300,), (5, 5), (17,)]
    params = [f32_exact(rng.normal(size=s)) for s in shapes]
    grads = [[f32_exact(rng.normal(size=s) * (2.0 if t % 2 else 0.5)) for s in shapes] for t in range(9)]
    W = 5
    hp = npo.Hyper(warmup=W, lambda_abs=12.0, lambda_rel=1.04, beta=0.9)
    hist, *_ = run(impl, params, grads, hp)
    clipped_steps = 0
    brute_min = None
    for t, (r, gs) in enumerate(zip(hist[:W], grads[:W]), start=1):
        assert len(set(np.asarray(r["h"]).tolist())) == 1 and len(set(np.asarray(r["flag"]).tolist())) == 1
        # textbook global-norm clipping (library routine; loose because of its 1e-6 in the denominator)
        ps = [torch.zeros(g.shape, dtype=torch.float64, requires_grad=True) for g in gs]
        for p, g in zip(ps, gs):
            p.grad = torch.tensor(g, dtype=torch.float64)
        total = float(torch.nn.utils.clip_grad_norm_(ps, hp.lambda_abs))
        assert float(r["global_norm"]) == pytest.approx(total, rel=1e-12)
        per = np.array([float(p.grad.norm()) for p in ps])
        np.testing.assert_allclose(r["clipped"], per, rtol=1e-6)
        clipped_steps += int(total > hp.lambda_abs)
        assert bool(r["flag"][0]) == (total > hp.lambda_abs)
        brute_min = per if brute_min is None else np.minimum(brute_min, per)
        np.testing.assert_allclose(np.asarray(r["gamma"], np.float64), brute_min, rtol=1e-6)
    assert 0 < clipped_steps < W                                 # both branches of the min{.,1} were taken
    # first AdaGC step: decisions are per tensor, taken against lambda_rel * (warm-up minimum)
    r = hist[W]
    n = np.array([np.linalg.norm(g.astype(np.float64)) for g in grads[W]])
    g_prev = np.asarray(hist[W - 1]["gamma"], np.float64)
    np.testing.assert_array_equal(r["flag"], n > hp.lambda_rel * g_prev)
    assert r["flag"].any()


def test_incoming_gamma_ignored_at_step_one_only():
    hp = npo.Hyper(warmup=0)
    garbage = np.array([123.0, np.nan], np.float32)
    for impl in IMPLS:
        r = impl.decisions([9.0, 16.0], garbage, 1, hp)
        np.testing.assert_array_equal(np.asarray(r["gamma"], np.float64), [3.0, 4.0])
        assert not np.asarray(r["flag"]).any()
        r = impl.decisions([9.0, 16.0], np.array([1.0, 8.0], np.float32), 2, hp)
        np.testing.assert_array_equal(np.asarray(r["flag"]), [True, False])


@pytest.mark.parametrize("impl", IMPLS, ids=lambda i: i.name)
def test_degenerate_norms(impl):
    hp = npo.Hyper(warmup=0, beta=0.5, lambda_rel=2.0)
    # zero gradient: never flagged, gamma decays
    r = impl.decisions([0.0], np.array([4.0], np.float32), 5, hp)
    assert not r["flag"][0] and r["h"][0] == 1.0 and float(r["gamma"][0]) == 2.0
    # zero gamma is absorbing: any non-zero gradient is clipped to zero (literal reading, no hidden epsilon)
    r = impl.decisions([4.0], np.array([0.0], np.float32), 5, hp)
    assert r["flag"][0] and r["h"][0] == 0.0 and float(r["gamma"][0]) == 0.0
    # equality is not a clip (strict >), and both readings give the same values
    r = impl.decisions([64.0], np.array([4.0], np.float32), 5, hp)
    assert not r["flag"][0] and r["h"][0] == 1.0 and float(r["gamma"][0]) == 0.5 * 4 + 0.5 * 8
    # non-finite norm: comparisons are false, h = 1, NaN propagates like in plain AdamW
    r = impl.decisions([float("nan")], np.array([4.0], np.float32), 5, hp)
    assert not r["flag"][0] and r["h"][0] == 1.0 and math.isnan(float(r["gamma"][0]))
    # warm-up with zero global norm
    hpw = npo.Hyper(warmup=3, lambda_abs=1.0)
    r = impl.decisions([0.0, 0.0], np.zeros(2, np.float32), 1, hpw)
    assert not np.asarray(r["flag"]).any() and (np.asarray(r["h"]) == 1.0).all()


# ----------------------------------------------------------------------------- the two oracles agree; brute force
def _brute_force(params, grads_per_step, hp):
    """Scalar Python loops, math.fsum for the sums, float64 state."""
    theta = [[float(x) for x in np.ravel(p)] for p in params]
    m = [[0.0] * len(p) for p in theta]
    v = [[0.0] * len(p) for p in theta]
    gamma = [0.0] * len(theta)
    flags = []
    for t, grads in enumerate(grads_per_step, start=1):
        gl = [[float(x) for x in np.ravel(g)] for g in grads]
        n = [math.sqrt(math.fsum(x * x for x in g)) for g in gl]
        if t <= hp.warmup:
            G = math.sqrt(math.fsum(x * x for g in gl for x in g))
            h = [min(hp.lambda_abs / G, 1.0) if G > 0 else 1.0] * len(gl)
            cn = [h[i] * n[i] for i in range(len(gl))]
            gamma = cn if t == 1 else [min(a, b) for a, b in zip(gamma, cn)]
            flags.append([G > hp.lambda_abs] * len(gl))
        else:
            if t == 1:
                gamma = list(n)
            h = [min(hp.lambda_rel * gamma[i] / n[i], 1.0) if n[i] > 0 else 1.0 for i in range(len(gl))]
            flags.append([n[i] > hp.lambda_rel * gamma[i] for i in range(len(gl))])
            gamma = [hp.beta * gamma[i] + (1 - hp.beta) * h[i] * n[i] for i in range(len(gl))]
        for i, g in enumerate(gl):
            for j, x in enumerate(g):
                gh = h[i] * x
                m[i][j] = hp.beta1 * m[i][j] + (1 - hp.beta1) * gh
                v[i][j] = hp.beta2 * v[i][j] + (1 - hp.beta2) * gh * gh
                mh = m[i][j] / (1 - hp.beta1 ** t)
                vh = v[i][j] / (1 - hp.beta2 ** t)
                theta[i][j] = theta[i][j] - hp.lr * hp.wd * theta[i][j] - hp.lr * mh / (math.sqrt(vh) + hp.eps)
    return theta, m, v, gamma, flags


def test_brute_force_tiny():
    rng = np.random.RandomState(11)
    shapes = [(4, 3), (5,), (2, 2)]
    params = [f32_exact(rng.normal(size=s)) for s in shapes]
    grads = []
    for t in range(12):
        gs = [f32_exact(rng.normal(size=s) * 1e-2) for s in shapes]
        if t == 7:
            gs[1] = gs[1] * np.float32(100)
        grads.append(gs)
    hp = npo.Hyper(lr=1e-2, warmup=3, lambda_abs=0.03, lambda_rel=1.05, beta=0.98)
    bth, bm, bv, bgam, bflags = _brute_force(params, grads, hp)
    # float64-state oracle: tight
    o = npo.AdaGCAdamW(params, hp, np.float64)
    for gs, bf in zip(grads, bflags):
        r = o.step(gs)
        np.testing.assert_array_equal(r.flag, bf)
    for a, b in zip(o.theta, bth):
        np.testing.assert_allclose(a.ravel(), b, rtol=1e-12)
    np.testing.assert_allclose(o.gamma, bgam, rtol=1e-12)
    assert any(any(f) for f in bflags[3:])
    # fp32-storage oracles: both, to storage precision
    for impl in IMPLS:
        hist, theta, m, v, gamma = run(impl, params, grads, hp)
        for r, bf in zip(hist, bflags):
            np.testing.assert_array_equal(np.asarray(r["flag"]), bf)
        for a, b in zip(theta, bth):
            np.testing.assert_allclose(a.ravel(), b, rtol=1e-5, atol=1e-7)
        np.testing.assert_allclose(gamma, bgam, rtol=1e-6)


def test_numpy_and_c_oracles_agree_on_a_random_layout():
    rng = np.random.RandomState(12)
    sizes = [1, 3, 7, 15, 16, 17, 64, 1000, 4099, 70001]
    off, o = [], 0
    for n in sizes:
        off.append(o)
        o += (n + 7) // 8 * 8
    theta0 = f32_exact(rng.normal(0, 0.02, size=o))
    hpd = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1, lambda_rel=1.04, beta=0.99,
               lambda_abs=0.05, warmup=3)
    hp = npo.Hyper(**hpd)
    A = co.ArenaOracle(off, sizes, theta0, **hpd)
    B = npo.AdaGCAdamW([theta0[a:a + n] for a, n in zip(off, sizes)], hp, np.float32)
    n_flags = 0
    for t in range(1, 16):
        g = f32_exact(rng.standard_t(2, size=o) * 1e-3)
        if t in (8, 11):
            g[off[7]:off[7] + sizes[7]] *= np.float32(300)
        ra = A.step(g)
        rb = B.step([g[a:a + n] for a, n in zip(off, sizes)])
        np.testing.assert_array_equal(ra["flag"], rb.flag)
        np.testing.assert_allclose(ra["h"], rb.h, rtol=1e-14)
        np.testing.assert_allclose(ra["gamma"], rb.gamma, rtol=1.2e-7)
        n_flags += int(rb.flag.sum())
    assert n_flags > 0
    np.testing.assert_array_equal(A.clip_count, B.clip_count)
    for i, (a, n) in enumerate(zip(off, sizes)):
        np.testing.assert_allclose(A.theta[a:a + n], B.theta[i], rtol=3e-7, atol=1e-10)
        np.testing.assert_allclose(A.m[a:a + n], B.m[i], rtol=3e-7, atol=1e-30)
        np.testing.assert_allclose(A.v[a:a + n], B.v[i], rtol=3e-7, atol=1e-30)


def test_storage_rounding_stays_close_to_float64_state():
    rng = np.random.RandomState(13)
    params = [rng.normal(0, 0.02, size=500).astype(np.float32)]
    hp = npo.Hyper(warmup=5, lambda_abs=0.01)
    a, b = npo.AdaGCAdamW(params, hp, np.float32), npo.AdaGCAdamW(params, hp, np.float64)
    for t in range(60):
        g = [f32_exact(rng.normal(0, 1e-3, size=500) * (40 if t == 30 else 1))]
        ra, rb = a.step(g), b.step(g)
        np.testing.assert_array_equal(ra.flag, rb.flag)
    np.testing.assert_allclose(a.theta[0], b.theta[0], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(a.gamma, b.gamma, rtol=1e-5)


def test_clip_only_scaling_in_gradient_dtype():
    rng = np.random.RandomState(14)
    g = torch.from_numpy(rng.standard_t(3, size=5000).astype(np.float32) * 1e-4).to(torch.bfloat16)
    bits = g.view(torch.int16).numpy().view(np.uint16).copy()
    h = 0.3712
    out = co.scale(bits, h)
    want64 = npo.clipped_grad(g.double().numpy(), h)
    got = torch.from_numpy(out.view(np.int16)).view(torch.bfloat16).double().numpy()
    # nearest bf16 to the float64 product: error at most half a bf16 ulp (<= 2^-8 relative)
    assert (np.abs(got - want64) <= np.abs(want64) * 2.0 ** -8 + 1e-45).all()
    gf = f32_exact(rng.normal(size=1000))
    np.testing.assert_array_equal(co.scale(gf, h), (h * gf.astype(np.float64)).astype(np.float32))


# ----------------------------------------------------------------------------- Lion on the clipped gradient
def _lion(impl_name, theta, g, m, h, lr, b1, b2, wd):
    if impl_name == "numpy":
        return npo.lion_update(theta, g, m, h, lr, b1, b2, wd, np.float32)
    th, mm = np.array(theta, np.float32), np.array(m, np.float32)
    co.lion_update(th, np.ascontiguousarray(g, np.float32), mm, h, lr, b1, b2, wd)
    return th, mm


@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_lion_closed_forms(impl_name):
    rng = np.random.RandomState(21)
    n = 300
    theta0 = f32_exact(rng.normal(size=n))
    g = f32_exact(rng.normal(size=n) * 1e-2)
    g[::7] = 0.0
    lr, b1, b2, wd = 1e-3, 0.9, 0.99, 0.1
    # first step from m = 0: c = (1-b1) h g, so the update is lr * sign(g); m_1 = (1-b2) h g
    for h in (1.0, 0.125):
        th, m = _lion(impl_name, theta0, g, np.zeros(n, np.float32), h, lr, b1, b2, wd)
        want = theta0.astype(np.float64) * (1 - lr * wd) - lr * np.sign(g.astype(np.float64))
        np.testing.assert_allclose(th, want, rtol=2e-7, atol=1e-9)
        np.testing.assert_allclose(m, (1 - b2) * h * g.astype(np.float64), rtol=2e-7)
    # constant gradient: m_t = g (1 - b2^t); theta_t = theta_0 r^t - lr s (1 - r^t)/(1 - r), r = 1 - lr wd
    th, m = theta0.copy(), np.zeros(n, np.float32)
    T = 50
    for _ in range(T):
        th, m = _lion(impl_name, th, g, m, 1.0, lr, b1, b2, wd)
    r = 1 - lr * wd
    sgn = np.sign(g.astype(np.float64))
    np.testing.assert_allclose(m, g.astype(np.float64) * (1 - b2 ** T), rtol=1e-5)
    np.testing.assert_allclose(th, theta0.astype(np.float64) * r ** T - lr * sgn * (1 - r ** T) / (1 - r),
                               rtol=1e-5, atol=1e-7)
    # the step size never depends on the gradient's magnitude: |theta_t - r theta_{t-1}| is lr or 0
    th2, _ = _lion(impl_name, theta0, g * np.float32(1e4), np.zeros(n, np.float32), 0.3, lr, b1, b2, wd)
    th1, _ = _lion(impl_name, theta0, g, np.zeros(n, np.float32), 1.0, lr, b1, b2, wd)
    np.testing.assert_array_equal(th1, th2)
    # sign follows the interpolation c, not the gradient: a small opposite gradient does not flip it
    m0 = np.full(4, 1.0, np.float32)
    gneg = np.full(4, -1.0, np.float32)
    th, m = _lion(impl_name, np.zeros(4, np.float32), gneg, m0, 1.0, lr, b1, b2, 0.0)
    np.testing.assert_allclose(th, -lr * np.ones(4), rtol=1e-6)          # c = 0.9 - 0.1 > 0
    th, m = _lion(impl_name, np.zeros(4, np.float32), gneg * np.float32(10), m0, 1.0, lr, b1, b2, 0.0)
    np.testing.assert_allclose(th, +lr * np.ones(4), rtol=1e-6)          # c = 0.9 - 1.0 < 0
    np.testing.assert_allclose(m, 0.99 * 1.0 + 0.01 * -10.0, rtol=1e-6)


def test_lion_brute_force_and_oracles_agree():
    rng = np.random.RandomState(22)
    n = 64
    theta = f32_exact(rng.normal(size=n)); m = np.zeros(n, np.float32)
    tb = [float(x) for x in theta]; mb = [0.0] * n
    tc, mc = theta.copy(), m.copy()
    lr, b1, b2, wd = 3e-4, 0.9, 0.99, 0.1
    for t in range(20):
        g = f32_exact(rng.standard_t(3, size=n) * 1e-2)
        h = 1.0 if t % 3 else 0.37
        theta, m = npo.lion_update(theta, g, m, h, lr, b1, b2, wd, np.float32)
        co.lion_update(tc, g, mc, h, lr, b1, b2, wd)
        for j in range(n):
            gh = h * float(g[j])
            c = b1 * mb[j] + (1 - b1) * gh
            tb[j] = tb[j] - lr * (math.copysign(1.0, c) * (c != 0) + wd * tb[j])
            mb[j] = b2 * mb[j] + (1 - b2) * gh
    np.testing.assert_allclose(theta, tb, rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(m, mb, rtol=1e-5, atol=1e-9)
    np.testing.assert_allclose(tc, theta, rtol=3e-7, atol=1e-9)
    np.testing.assert_allclose(mc, m, rtol=3e-7, atol=1e-12)


# ----------------------------------------------------------------------------- ablation variants (Section 5)
def _decide(impl_name, s, gamma, step, hp, **kw):
    if impl_name == "numpy":
        r = npo.clip_decisions(s, gamma, step, hp, np.float32, **kw)
        return dict(h=r.h, flag=r.flag, gamma=np.asarray(r.gamma, np.float32), norm=r.norm)
    g = np.array(gamma, np.float32)
    r = co.clip_decisions(np.asarray(s, np.float64), g, step, hp.lambda_rel, hp.beta, hp.lambda_abs, hp.warmup, **kw)
    return dict(h=r["h"], flag=r["flag"], gamma=g, norm=r["norm"])


@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_global_adaptive_is_the_algorithm_on_the_concatenated_gradient(impl_name):
    """'Global AdaGC' (one adaptive threshold for the whole model) must equal the per-tensor algorithm run on
    the single tensor made of all gradients; the T = 1 run below uses the plain (non-variant) code path."""
    rng = np.random.RandomState(31)
    sizes = [40, 1000, 7, 333]
    hp = npo.Hyper(warmup=3, lambda_abs=0.08, lambda_rel=1.04, beta=0.9)
    gam_g = np.zeros(len(sizes), np.float32)
    gam_1 = np.zeros(1, np.float32)
    seen = set()
    for t in range(1, 16):
        gs = [f32_exact(rng.normal(size=n) * 1e-3 * (30 if t in (7, 11) else 1)) for n in sizes]
        s = [npo.sumsq(g) for g in gs]
        one = _decide(impl_name, [npo.sumsq(np.concatenate(gs))], gam_1, t, hp)
        glo = _decide(impl_name, s, gam_g, t, hp, global_adaptive=True)
        gam_1, gam_g = one["gamma"], glo["gamma"]
        assert len(set(np.asarray(glo["h"]).tolist())) == 1 and len(set(np.asarray(glo["flag"]).tolist())) == 1
        assert bool(glo["flag"][0]) == bool(one["flag"][0])
        assert glo["h"][0] == pytest.approx(one["h"][0], rel=1e-14)
        np.testing.assert_allclose(gam_g, np.full(len(sizes), gam_1[0]), rtol=1.2e-7)
        np.testing.assert_allclose(glo["norm"], [math.sqrt(x) for x in s], rtol=1e-15)
        seen.add((t <= hp.warmup, bool(one["flag"][0])))
    assert (False, True) in seen and (False, False) in seen          # AdaGC steps both clipped and calm


@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_keep_initial_uses_the_callers_gamma_from_the_first_step(impl_name):
    """Constant initialization of the ablation: gamma_0 given by the caller, no seeding at t = 1."""
    hp = npo.Hyper(warmup=0, lambda_rel=2.0, beta=0.5)
    r = _decide(impl_name, [9.0, 16.0], np.array([1.0, 8.0], np.float32), 1, hp, keep_initial=True)
    np.testing.assert_array_equal(np.asarray(r["flag"]), [True, False])     # 3 > 2*1 ; 4 <= 2*8
    np.testing.assert_array_equal(np.asarray(r["h"]), [2.0 / 3.0, 1.0])
    np.testing.assert_array_equal(r["gamma"], np.array([0.5 * 1 + 0.5 * 2, 0.5 * 8 + 0.5 * 4], np.float32))
    # default behaviour for comparison: seeded with the norms, nothing clipped
    r0 = _decide(impl_name, [9.0, 16.0], np.array([1.0, 8.0], np.float32), 1, hp)
    assert not np.asarray(r0["flag"]).any() and list(r0["gamma"]) == [3.0, 4.0]
    # warm-up with keep_initial: running minimum starts from the caller's value
    hpw = npo.Hyper(warmup=5, lambda_abs=100.0)
    r = _decide(impl_name, [9.0, 16.0], np.array([1.0, 8.0], np.float32), 1, hpw, keep_initial=True)
    assert list(r["gamma"]) == [1.0, 4.0]
    # after the first step the variant changes nothing
    a = _decide(impl_name, [9.0, 16.0], np.array([1.0, 8.0], np.float32), 4, hp, keep_initial=True)
    b = _decide(impl_name, [9.0, 16.0], np.array([1.0, 8.0], np.float32), 4, hp)
    np.testing.assert_array_equal(a["gamma"], b["gamma"])


@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_thresholded_initialization_hand_values_and_special_cases(impl_name):
    """Thresholded initialization of the ablation (variant 3, gamma_t,i = min(||g_t,i||, cap), cap 0.1 there):
    the constant takes the place of gamma_t-1,i in the warm-up line, so the value after warm-up is
    min(last warm-up clipped norm, cap) and earlier warm-up steps leave no trace."""
    hp = npo.Hyper(warmup=3, lambda_abs=100.0, lambda_rel=2.0, beta=0.5)         # no warm-up clipping: hat(g) = g
    gam = np.array([np.nan, np.nan], np.float32)                                  # incoming content is irrelevant
    seq = [([25.0, 144.0], [5.0, 6.0]),       # norms 5, 12; cap 6 -> 5, 6
           ([49.0, 9.0], [6.0, 3.0]),         # norms 7, 3 -> 6, 3: NOT min with the previous 5 (no running minimum)
           ([1.0, 100.0], [1.0, 6.0])]        # norms 1, 10 -> 1, 6
    for t, (s, want) in enumerate(seq, start=1):
        r = _decide(impl_name, s, gam, t, hp, ema_cap=6.0)
        gam = r["gamma"]
        assert list(gam) == want and not np.asarray(r["flag"]).any()
    # first AdaGC step uses what the last warm-up step left: thresholds 2*1 and 2*6
    r = _decide(impl_name, [16.0, 100.0], gam, 4, hp, ema_cap=6.0)
    np.testing.assert_array_equal(np.asarray(r["flag"]), [True, False])            # 4 > 2 ; 10 <= 12
    np.testing.assert_array_equal(r["gamma"], np.array([0.5 * 1 + 0.5 * 2, 0.5 * 6 + 0.5 * 10], np.float32))
    # warm-up clipping active: the capped quantity is the CLIPPED norm h_t ||g_t,i|| (Algorithm 1 writes the hat)
    hpc = npo.Hyper(warmup=3, lambda_abs=6.5, lambda_rel=2.0, beta=0.5)           # G = 13 -> h = 0.5
    r = _decide(impl_name, [25.0, 144.0], np.zeros(2, np.float32), 1, hpc, ema_cap=4.0)
    assert list(r["gamma"]) == [2.5, 4.0] and list(np.asarray(r["h"])) == [0.5, 0.5]
    # T_start = 0: the seed of step 1 is capped, then Eq. 3 applies to it
    hp0 = npo.Hyper(warmup=0, lambda_rel=2.0, beta=0.5)
    r = _decide(impl_name, [9.0, 16.0], np.zeros(2, np.float32), 1, hp0, ema_cap=1.5)
    np.testing.assert_array_equal(np.asarray(r["flag"]), [False, True])            # 3 <= 2*1.5 ; 4 > 2*1.5
    np.testing.assert_array_equal(r["gamma"], np.array([0.5 * 1.5 + 0.5 * 3, 0.5 * 1.5 + 0.5 * 3], np.float32))
    # special cases that reduce to the default: one warm-up step with a cap nothing reaches (the seed IS the clipped
    # norm), and any AdaGC step after the first (the variant only touches seeding and warm-up)
    rng = np.random.RandomState(5)
    s = (rng.standard_t(3, size=50) ** 2 + 1e-3).tolist()
    hp1 = npo.Hyper(warmup=1, lambda_abs=0.7)
    a = _decide(impl_name, s, np.zeros(50, np.float32), 1, hp1, ema_cap=1e30)
    b = _decide(impl_name, s, np.zeros(50, np.float32), 1, hp1)
    np.testing.assert_array_equal(a["gamma"], b["gamma"])
    g0 = np.abs(rng.normal(size=50)).astype(np.float32)
    a = _decide(impl_name, s, g0.copy(), 9, hp1, ema_cap=0.1)
    b = _decide(impl_name, s, g0.copy(), 9, hp1)
    np.testing.assert_array_equal(a["gamma"], b["gamma"])
    np.testing.assert_array_equal(np.asarray(a["flag"]), np.asarray(b["flag"]))


def test_thresholded_initialization_brute_force_and_oracles_agree():
    """gamma after warm-up = min(h_T ||g_T,i||, cap) for the LAST warm-up step T (brute force over a random run),
    never above the cap; numpy and C oracles agree bit for bit on gamma and flags."""
    rng = np.random.RandomState(77)
    T, W, cap = 40, 6, 0.1
    hp = npo.Hyper(warmup=W, lambda_abs=1.0, lambda_rel=1.04, beta=0.99)
    gn, gc = np.zeros(T, np.float32), np.zeros(T, np.float32)
    for t in range(1, W + 5):
        s = (np.abs(rng.standard_t(2, size=T)) * 0.05) ** 2
        rn = _decide("numpy", s.tolist(), gn, t, hp, ema_cap=cap)
        rc = _decide("c", s.tolist(), gc, t, hp, ema_cap=cap)
        gn, gc = rn["gamma"], rc["gamma"]
        np.testing.assert_array_equal(gn, gc)
        np.testing.assert_array_equal(np.asarray(rn["flag"]), np.asarray(rc["flag"]))
        if t <= W:
            G = math.sqrt(float(np.sum(s)))
            h = min(1.0 / G, 1.0)
            want = np.minimum(h * np.sqrt(s), cap).astype(np.float32)
            np.testing.assert_array_equal(gn, want)
            assert (gn <= np.float32(cap)).all()


# ----------------------------------------------------------------------------- SGD with momentum on the clipped gradient
@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_sgdm_matches_library_sgd(impl_name):
    """Special case that reduces to a library routine: torch.optim.SGD(momentum, weight_decay) fed the
    clipped gradients, float64."""
    rng = np.random.RandomState(41)
    n = 200
    theta0 = f32_exact(rng.normal(size=n))
    lr, mu, wd = 1e-2, 0.9, 0.05
    p = torch.tensor(theta0.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, weight_decay=wd)
    th, m = theta0.copy(), np.zeros(n, np.float32)
    for t in range(25):
        g = f32_exact(rng.standard_t(3, size=n) * 1e-2)
        h = 1.0 if t % 4 else 0.21
        p.grad = torch.tensor(h * g.astype(np.float64))
        opt.step()
        if impl_name == "numpy":
            th, m = npo.sgdm_update(th, g, m, h, lr, mu, wd, np.float32)
        else:
            co.sgdm_update(th, g, m, h, lr, mu, wd)
    np.testing.assert_allclose(th, p.detach().numpy(), rtol=2e-6, atol=1e-7)      # fp32 storage vs float64 library run
    th64, m64 = theta0.astype(np.float64), np.zeros(n)
    p2 = torch.tensor(theta0.astype(np.float64), requires_grad=True)
    opt2 = torch.optim.SGD([p2], lr=lr, momentum=mu, weight_decay=wd)
    rng = np.random.RandomState(42)
    for t in range(25):
        g = rng.normal(size=n)
        p2.grad = torch.tensor(0.5 * g)
        opt2.step()
        th64, m64 = npo.sgdm_update(th64, g, m64, 0.5, lr, mu, wd, np.float64)
    np.testing.assert_allclose(th64, p2.detach().numpy(), rtol=1e-12, atol=1e-15)
