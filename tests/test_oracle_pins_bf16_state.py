"""Pins for the oracles' bfloat16-stored optimizer state (m and v kept as bfloat16, fp32 master theta).

The paper trains in bfloat16 / float8 precision (Appendix "Hyper-Parameters") and does not say how stored
optimizer state is rounded.  Reading pinned here: a step reads the stored bfloat16 moments exactly, computes
in float64, updates theta from the UNROUNDED new moments, and rounds the moments to the nearest bfloat16
(ties to even) when it stores them.

Nothing here touches the CUDA path.  The pins are the library's own conversion (torch .to(bfloat16) on
fp32-exact inputs), torch.optim.AdamW / SGD in float64 started from a given state, the definition of
"nearest representable value", a derived stall bound for a constant gradient, and numpy-vs-C agreement.
"""
import numpy as np
import pytest
import torch

from oracle import adagc_oracle as npo
from oracle import c_oracle as co


def bits_to_f64(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bits(x):
    """bit patterns of float32 values that are exactly bfloat16 values"""
    u = np.asarray(x, np.float32).view(np.uint32)
    assert (u & 0xFFFF == 0).all(), "value is not representable in bfloat16"
    return (u >> 16).astype(np.uint16)


def spacing_bf16(x):
    """distance between neighbouring bfloat16 values around x (from the format: 8 significand bits)"""
    x = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.maximum(x, 2.0 ** -126)))
    return 2.0 ** (np.maximum(e, -126) - 7)


def assert_is_nearest_bf16(stored, exact, what):
    """`stored` holds bfloat16 values and none of its neighbours is closer to `exact`."""
    stored, exact = np.asarray(stored, np.float64), np.asarray(exact, np.float64)
    assert (stored.astype(np.float32).view(np.uint32) & 0xFFFF == 0).all(), f"{what}: not a bfloat16 value"
    # neighbouring bfloat16 values around `exact` are one spacing (of exact's binade) apart
    assert (np.abs(stored - exact) <= 0.5 * spacing_bf16(exact) * (1 + 1e-12)).all(), f"{what}: not the nearest bfloat16"


class NumpyBF:
    name = "numpy"

    @staticmethod
    def adamw(theta, g, m, v, h, step, hp):
        """m, v: float arrays of bfloat16 values.  Returns theta (fp32), m, v (float64 views of the stored values)."""
        th, m1, v1 = npo.adamw_update(theta, g, m, v, h, step, hp, np.float32, moment_dtype="bf16")
        return th, m1.astype(np.float64), v1.astype(np.float64)


class CBF:
    name = "c"

    @staticmethod
    def adamw(theta, g, m, v, h, step, hp):
        th = np.array(theta, np.float32)
        mb, vb = f32_to_bits(m), f32_to_bits(v)
        co.adamw_update_bf16state(th, np.ascontiguousarray(g, np.float32), mb, vb, h, step, hp.lr, hp.beta1,
                                  hp.beta2, hp.eps, hp.wd)
        return th, bits_to_f64(mb), bits_to_f64(vb)


BF_IMPLS = [NumpyBF, CBF]


def bf16_values(rng, n, scale):
    """random values that are exactly bfloat16 values (via the library's conversion of fp32 numbers)"""
    x = torch.from_numpy((rng.standard_normal(n) * scale).astype(np.float32))
    return x.to(torch.bfloat16).to(torch.float32).numpy()


# ----------------------------------------------------------------------------- the rounding itself
def test_rounding_matches_the_library_conversion_and_ties_go_to_even():
    rng = np.random.RandomState(3)
    x = np.concatenate([rng.standard_normal(200000) * 10.0 ** rng.uniform(-44, 38, 200000),
                        [0.0, -0.0, 1.0, -1.0, 3.3895e38, 3.4e38, -3.4e38, 1e-40, 2.0 ** -133, 2.0 ** -134,
                         1.5 * 2.0 ** -133, np.inf, -np.inf]]).astype(np.float32)
    # exact ties: midpoints between neighbouring bfloat16 values, even and odd lower neighbours, both signs
    lows = np.array([0x3F80, 0x3F81, 0x4000, 0x40FF, 0x0001, 0x0002, 0x7F7E, 0x0080, 0x007F], np.uint32)
    mids = ((lows << 16) | 0x8000).view(np.float32)
    x = np.concatenate([x, mids, -mids])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()         # fp32 -> bf16: one rounding
    got_np = npo.round_to_bf16(x.astype(np.float64))
    assert np.array_equal(got_np.astype(np.float32).view(np.uint32), want.view(np.uint32))
    got_c = np.array([co.double_to_bf16_bits(float(v)) for v in x[-5000:]], np.uint16)
    assert np.array_equal(got_c, (want[-5000:].view(np.uint32) >> 16).astype(np.uint16))
    # the tie cases really are ties and went to the even neighbour
    tie_bits = (want[-2 * len(lows):-len(lows)].view(np.uint32) >> 16)
    assert (tie_bits % 2 == 0).all() and np.array_equal(tie_bits, lows + (lows & 1))
    assert np.isnan(npo.round_to_bf16(np.array([np.nan]))[0])


def test_rounding_margin_is_the_distance_to_a_flip():
    """bf16_rounding_margin: 0 at a midpoint, half the spacing at a bfloat16 value (a quarter at a power of two, whose
    lower neighbours are twice as dense), and any perturbation smaller than margin * scale leaves the rounding
    unchanged while a slightly larger one (towards the nearer flip) changes it."""
    assert npo.bf16_rounding_margin(np.array([1.0 + 2.0 ** -8]), 1.0)[0] == 0.0
    assert npo.bf16_rounding_margin(np.array([1.0 + 2.0 ** -7]), 1.0)[0] == 2.0 ** -8
    assert npo.bf16_rounding_margin(np.array([1.0]), 1.0)[0] == 2.0 ** -9
    assert npo.bf16_rounding_margin(np.array([3.0]), 2.0)[0] == 2.0 ** -7 / 2.0
    rng = np.random.RandomState(4)
    x = rng.standard_normal(20000) * 10.0 ** rng.uniform(-30, 30, 20000)
    d = npo.bf16_rounding_margin(x, 1.0)
    r0 = npo.round_to_bf16(x)
    for sgn in (-1.0, 1.0):
        assert np.array_equal(npo.round_to_bf16(x + sgn * 0.999 * d), r0)
    flipped = (npo.round_to_bf16(x + 1.001 * d) != r0) | (npo.round_to_bf16(x - 1.001 * d) != r0)
    assert flipped.all()


# ----------------------------------------------------------------------------- one step against the library
@pytest.mark.parametrize("impl", BF_IMPLS, ids=lambda i: i.name)
@pytest.mark.parametrize("step", [1, 2, 7, 100])
def test_one_step_from_a_given_state_matches_library_adamw(impl, step):
    """torch.optim.AdamW (float64) started from the same theta, m, v and step count: theta agrees (so theta was
    updated from the unrounded moments), and the stored moments are the bfloat16 values nearest to the library's."""
    rng = np.random.RandomState(100 + step)
    n = 4096
    hp = npo.Hyper(lr=3e-3, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)
    theta0 = (rng.standard_normal(n) * 0.5).astype(np.float32)
    g = (rng.standard_t(3, size=n) * 1e-2).astype(np.float32)
    h = 0.37
    if step == 1:
        m0, v0 = np.zeros(n, np.float32), np.zeros(n, np.float32)
    else:
        m0 = bf16_values(rng, n, 1e-2)
        v0 = bf16_values(rng, n, 1e-2) ** 2
        v0 = torch.from_numpy(v0).to(torch.bfloat16).to(torch.float32).numpy()
    p = torch.tensor(theta0.astype(np.float64), requires_grad=True)
    opt = torch.optim.AdamW([p], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.eps, weight_decay=hp.wd, foreach=False)
    opt.state[p] = {"step": torch.tensor(float(step - 1)), "exp_avg": torch.tensor(m0.astype(np.float64)),
                    "exp_avg_sq": torch.tensor(v0.astype(np.float64))}
    p.grad = torch.tensor(h * g.astype(np.float64))
    opt.step()
    th, m1, v1 = impl.adamw(theta0, g, m0, v0, h, step, hp)
    np.testing.assert_allclose(th, p.detach().numpy(), rtol=1.2e-7, atol=1e-30)           # fp32 storage of theta only
    assert_is_nearest_bf16(m1, opt.state[p]["exp_avg"].numpy(), "m")
    assert_is_nearest_bf16(v1, opt.state[p]["exp_avg_sq"].numpy(), "v")
    assert (m1 != opt.state[p]["exp_avg"].numpy()).mean() > 0.9, "the moments were not rounded at all"


@pytest.mark.parametrize("impl", BF_IMPLS, ids=lambda i: i.name)
def test_theta_is_the_fp32_state_paths_theta_bit_for_bit(impl):
    """Rounding happens on store only: from the same stored inputs the step's theta equals, bit for bit, the theta of
    the (separately pinned) fp32-state update, and the stored moments are the nearest bfloat16 of its float64 moments."""
    rng = np.random.RandomState(8)
    n = 3000
    hp = npo.Hyper(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-15, wd=0.05)
    theta0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    m0, v0 = bf16_values(rng, n, 1e-4), bf16_values(rng, n, 1e-8).__abs__()
    g = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    th, m1, v1 = impl.adamw(theta0, g, m0, v0, 1.0, 5, hp)
    th_ref, _, _ = npo.adamw_update(theta0, g, m0, v0, 1.0, 5, hp, np.float32)
    _, m64, v64 = npo.adamw_update(theta0, g, m0, v0, 1.0, 5, hp, np.float64)
    assert np.array_equal(th.view(np.uint32), th_ref.view(np.uint32))
    assert_is_nearest_bf16(m1, m64, "m")
    assert_is_nearest_bf16(v1, v64, "v")


# ----------------------------------------------------------------------------- an invariant of the iteration
@pytest.mark.parametrize("impl", BF_IMPLS, ids=lambda i: i.name)
def test_constant_gradient_stalls_within_the_derived_bound(impl):
    """With a constant gradient the fp32-state moments converge to g and g^2.  Stored as bfloat16 the iteration
    x <- round(beta x + (1 - beta) c) stops moving once the increment (1 - beta)|c - x| is below half the spacing, so
    it ends within spacing / (2 (1 - beta)) of the fixed point (plus one spacing for the last rounding), and approaches
    it monotonically.  beta1 = 0.9: 5 spacings; beta2 = 0.95: 10 spacings."""
    rng = np.random.RandomState(9)
    n = 512
    hp = npo.Hyper(lr=0.0, beta1=0.9, beta2=0.95, wd=0.0)
    g = (np.abs(rng.standard_normal(n)) * 1e-3 + 1e-4).astype(np.float32)
    theta = np.zeros(n, np.float32)
    m, v = np.zeros(n, np.float32), np.zeros(n, np.float32)
    prev_m, prev_v = m.astype(np.float64), v.astype(np.float64)
    for t in range(1, 301):
        theta, m, v = impl.adamw(theta, g, m.astype(np.float32), v.astype(np.float32), 1.0, t, hp)
        assert (m >= prev_m).all() and (v >= prev_v).all()            # monotone approach from below
        prev_m, prev_v = m, v
    g64 = g.astype(np.float64)
    assert (np.abs(m - g64) <= spacing_bf16(g64) * (0.5 / (1 - hp.beta1) + 1.0)).all()
    assert (np.abs(v - g64 ** 2) <= spacing_bf16(g64 ** 2) * (0.5 / (1 - hp.beta2) + 1.0)).all()
    assert (m <= g64 * (1 + 2.0 ** -8)).all() and (v <= g64 ** 2 * (1 + 2.0 ** -8)).all()   # never beyond the fixed point's rounding
    # the bound is not vacuous: some elements do stall short of the fixed point's own rounding
    assert (np.abs(m - g64) > spacing_bf16(g64)).any()


# ----------------------------------------------------------------------------- Lion and momentum SGD
@pytest.mark.parametrize("impl_name", ["numpy", "c"])
def test_lion_and_sgdm_store_the_nearest_bf16_and_leave_theta_alone(impl_name):
    rng = np.random.RandomState(10)
    n = 2048
    theta0 = (rng.standard_normal(n) * 0.02).astype(np.float32)
    m0 = bf16_values(rng, n, 1e-3)
    g = (rng.standard_t(3, size=n) * 1e-3).astype(np.float32)
    h, lr, b1, b2, wd, mu = 0.5, 1e-4, 0.9, 0.99, 0.1, 0.9
    # Lion
    th_ref, _ = npo.lion_update(theta0, g, m0, h, lr, b1, b2, wd, np.float32)
    _, m64 = npo.lion_update(theta0, g, m0, h, lr, b1, b2, wd, np.float64)
    if impl_name == "numpy":
        th, m1 = npo.lion_update(theta0, g, m0, h, lr, b1, b2, wd, np.float32, moment_dtype="bf16")
        m1 = m1.astype(np.float64)
    else:
        th, mb = theta0.copy(), f32_to_bits(m0)
        co.lion_update(th, g, mb, h, lr, b1, b2, wd)
        m1 = bits_to_f64(mb)
    assert np.array_equal(th.view(np.uint32), th_ref.view(np.uint32))
    assert_is_nearest_bf16(m1, m64, "Lion m")
    # momentum SGD, against the library started from the given momentum buffer
    p = torch.tensor(theta0.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, weight_decay=wd)
    opt.state[p] = {"momentum_buffer": torch.tensor(m0.astype(np.float64))}
    p.grad = torch.tensor(h * g.astype(np.float64))
    opt.step()
    if impl_name == "numpy":
        th, m1 = npo.sgdm_update(theta0, g, m0, h, lr, mu, wd, np.float32, moment_dtype="bf16")
        m1 = m1.astype(np.float64)
    else:
        th, mb = theta0.copy(), f32_to_bits(m0)
        co.sgdm_update(th, g, mb, h, lr, mu, wd)
        m1 = bits_to_f64(mb)
    np.testing.assert_allclose(th, p.detach().numpy(), rtol=1.2e-7, atol=1e-30)           # theta saw the unrounded momentum
    assert_is_nearest_bf16(m1, opt.state[p]["momentum_buffer"].numpy(), "SGD m")


# ----------------------------------------------------------------------------- the two oracles against each other
def test_numpy_and_c_oracles_agree_with_bf16_state_over_many_steps():
    """Whole path on a small ragged layout: decisions, gamma, theta and the stored moments, bit for bit."""
    rng = np.random.RandomState(11)
    sizes = [7, 300, 4097, 33]
    offs, o = [], 0
    for s in sizes:
        offs.append(o)
        o += (s + 7) // 8 * 8
    hp = npo.Hyper(lr=1e-3, warmup=3, lambda_abs=0.02, lambda_rel=1.04, beta=0.98)
    theta0 = (rng.standard_normal(o) * 0.02).astype(np.float32)
    ref_np = npo.AdaGCAdamW([theta0[a:a + s] for a, s in zip(offs, sizes)], hp, np.float32, moment_dtype="bf16")
    ref_c = co.ArenaOracle(offs, sizes, theta0, lr=hp.lr, beta1=hp.beta1, beta2=hp.beta2, eps=hp.eps, wd=hp.wd,
                           lambda_rel=hp.lambda_rel, beta=hp.beta, lambda_abs=hp.lambda_abs, warmup=hp.warmup,
                           bf16_state=True, tie_tol=1e-6)
    for t in range(1, 16):
        g = (rng.standard_t(3, size=o) * 1e-3 * (30.0 if t == 9 else 1.0)).astype(np.float32)
        r_np = ref_np.step([g[a:a + s] for a, s in zip(offs, sizes)])
        r_c = ref_c.step(g)
        assert np.array_equal(r_np.flag, r_c["flag"])
        np.testing.assert_allclose(r_np.gamma, r_c["gamma"], rtol=1e-7)
    for i, (a, s) in enumerate(zip(offs, sizes)):
        np.testing.assert_allclose(ref_np.theta[i], ref_c.theta[a:a + s], rtol=2e-7, atol=1e-12)
        same_m = f32_to_bits(ref_np.m[i]) == ref_c.m[a:a + s]
        same_v = f32_to_bits(ref_np.v[i]) == ref_c.v[a:a + s]
        # pow() and ** may differ in the last bit of a float64 coefficient; only an element that the C oracle itself
        # reports as decided within 1e-6 of a flip may round differently
        assert (same_m | (ref_c.ties[a:a + s] > 0)).all() and (same_v | (ref_c.ties[a:a + s] > 0)).all()
    assert ref_c.ties.mean() < 0.05


def test_c_oracle_counts_decisions_close_to_a_flip():
    """near_tie is incremented exactly for elements whose new m (or v) is within tie_tol of a rounding flip."""
    hp = npo.Hyper(lr=0.0, beta1=0.5, beta2=0.5, wd=0.0)
    # m1 = 0.5 * m0 + 0.5 * g: choose m0 = 1, g = 1 + 2^-6 -> m1 = 1 + 2^-7 ... a bfloat16 value (margin = half a spacing);
    # g = 1 + 2^-7 -> m1 = 1 + 2^-8: exactly the midpoint between 1 and 1 + 2^-7 (margin 0)
    m0 = np.array([1.0, 1.0, 1.0], np.float32)
    g = np.array([1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -7 + 2.0 ** -20], np.float32)
    v0 = np.zeros(3, np.float32)
    th, mb, vb, ties = np.zeros(3, np.float32), f32_to_bits(m0), f32_to_bits(v0), np.zeros(3, np.uint8)
    co.adamw_update_bf16state(th, g, mb, vb, 1.0, 3, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.wd, near_tie=ties, tie_tol=1e-5)
    assert ties.tolist() == [0, 1, 1]
    assert bits_to_f64(mb).tolist() == [1.0 + 2.0 ** -7, 1.0, 1.0 + 2.0 ** -7]     # tie to even; just above the midpoint rounds up
    _, _, _, mm, _ = npo.adamw_update(th, g, m0, v0, 1.0, 3, hp, np.float32, moment_dtype="bf16", return_margin=True)
    assert mm[1] == 0.0 and mm[0] > 1e-3 and 0 < mm[2] < 1e-5


# ----------------------------------------------------------------------------- the rounding decision taken in fp32
def _round_fraction(x, sig_bits, e_min):
    """Exact rational x -> nearest binary floating-point number with `sig_bits` significand bits and least exponent
    e_min for the last place (round half to even), returned as a Fraction."""
    from fractions import Fraction
    if x == 0:
        return Fraction(0)
    e = 0
    ax = abs(x)
    while ax >= Fraction(2) ** (e + 1):
        e += 1
    while ax < Fraction(2) ** e:
        e -= 1
    ulp_e = max(e - (sig_bits - 1), e_min)
    n = round(x / Fraction(2) ** ulp_e)                     # Python rounds halves to even
    return n * Fraction(2) ** ulp_e


def test_fp32_decision_follows_the_stated_single_precision_order_exactly():
    """The stored bfloat16 of the C oracle's fp32-decision mode equals, bit for bit, the stated formula evaluated in
    exact rational arithmetic with one rounding to single precision per operation (24 bits, last place >= 2^-149)
    and one rounding to bfloat16 (8 bits, last place >= 2^-133) at the end."""
    from fractions import Fraction as F
    rng = np.random.RandomState(21)
    n = 1500
    g = bf16_values(rng, n, 1e-4).astype(np.float32)
    g[:50] = (rng.standard_normal(50) * 1e-4).astype(np.float32)            # and some full-precision gradients
    m0, v0 = bf16_values(rng, n, 3e-5), np.abs(bf16_values(rng, n, 1e-8))
    theta = (rng.standard_normal(n) * 0.02).astype(np.float32)
    h, b1, b2 = 0.731, 0.9, 0.95
    f32 = lambda x: _round_fraction(x, 24, -149)
    bf = lambda x: _round_fraction(x, 8, -133)
    hf, b1f, o1f, b2f, o2f = (F(float(np.float32(x))) for x in (h, b1, 1.0 - b1, b2, 1.0 - b2))
    want_m, want_v = [], []
    for j in range(n):
        gh = f32(hf * F(float(g[j])))
        want_m.append(float(bf(f32(b1f * F(float(m0[j])) + f32(o1f * gh)))))
        want_v.append(float(bf(f32(b2f * F(float(v0[j])) + f32(o2f * f32(gh * gh))))))
    mb, vb = f32_to_bits(m0), f32_to_bits(v0)
    co.adamw_update_bf16state(theta.copy(), g, mb, vb, h, 3, 1e-3, b1, b2, 1e-8, 0.1, fp32_decision=True)
    assert np.array_equal(bits_to_f64(mb), np.array(want_m)) and np.array_equal(bits_to_f64(vb), np.array(want_v))
    # Lion's and momentum SGD's stored momentum, the same way
    mb = f32_to_bits(m0)
    co.lion_update(theta.copy(), g, mb, h, 1e-4, 0.9, 0.99, 0.1, fp32_decision=True)
    b2l, o2l = F(float(np.float32(0.99))), F(float(np.float32(1.0 - 0.99)))
    want = [float(bf(f32(b2l * F(float(m0[j])) + f32(o2l * f32(hf * F(float(g[j]))))))) for j in range(n)]
    assert np.array_equal(bits_to_f64(mb), np.array(want))
    mb = f32_to_bits(m0)
    co.sgdm_update(theta.copy(), g, mb, h, 1e-2, 0.9, 0.05, fp32_decision=True)
    muf, wdf = F(float(np.float32(0.9))), F(float(np.float32(0.05)))
    want = [float(bf(f32(muf * F(float(m0[j])) + f32(wdf * F(float(theta[j])) + f32(hf * F(float(g[j]))))))) for j in range(n)]
    assert np.array_equal(bits_to_f64(mb), np.array(want))


def test_fp32_and_float64_decisions_differ_only_at_reported_ties_and_by_one_neighbour():
    """The single-precision decision is pinned to the (library-pinned) float64 one: the stored values agree except
    where the float64 oracle itself reports that the rounding was decided within 1e-6 of a flip, and there they are
    neighbours.  With bfloat16 g and m and beta1 = 0.9 such ties are frequent: the float64 value is an exact decimal
    tie (x.5 spacings) for a few percent of the elements, which is why the decision must name its precision."""
    rng = np.random.RandomState(22)
    n = 200000
    g = bf16_values(rng, n, 1e-4).astype(np.float32)
    m0, v0 = bf16_values(rng, n, 3e-5), np.abs(bf16_values(rng, n, 1e-8))
    theta = (rng.standard_normal(n) * 0.02).astype(np.float32)
    th64, th32 = theta.copy(), theta.copy()
    m64, v64, m32, v32 = f32_to_bits(m0), f32_to_bits(v0), f32_to_bits(m0), f32_to_bits(v0)
    ties = np.zeros(n, np.uint8)
    co.adamw_update_bf16state(th64, g, m64, v64, 1.0, 4, 3e-4, 0.9, 0.95, 1e-8, 0.1, near_tie=ties, tie_tol=1e-6)
    co.adamw_update_bf16state(th32, g, m32, v32, 1.0, 4, 3e-4, 0.9, 0.95, 1e-8, 0.1, fp32_decision=True)
    assert np.array_equal(th64, th32)                                  # theta never sees the rounding decision
    m_terms = np.abs(0.9 * m0.astype(np.float64)) + np.abs(0.1 * g.astype(np.float64))
    for a, b, terms in ((m64, m32, m_terms), (v64, v32, None)):
        diff = a != b
        assert (~diff | (ties > 0)).all()
        # neighbours (bfloat16 bit patterns of one sign are ordered like the magnitudes they encode) -- or, where the
        # two terms of m' cancel completely, two different roundings of what is zero in exact arithmetic
        near = np.abs(a[diff].astype(np.int64) - b[diff].astype(np.int64)) == 1
        if terms is not None:
            near |= np.maximum(np.abs(bits_to_f64(a[diff])), np.abs(bits_to_f64(b[diff]))) <= 1e-6 * terms[diff]
        assert near.all()
    assert 0.01 < (ties > 0).mean() < 0.10 and (m64 != m32).mean() > 0.005
    # with full-precision fp32 gradients the ties are as rare as for arbitrary numbers
    g2 = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    ties2 = np.zeros(n, np.uint8)
    co.adamw_update_bf16state(theta.copy(), g2, f32_to_bits(m0), f32_to_bits(v0), 1.0, 4, 3e-4, 0.9, 0.95, 1e-8, 0.1,
                              near_tie=ties2, tie_tol=1e-6)
    assert (ties2 > 0).mean() < 4e-3


# ----------------------------------------------------------------------------- stochastic rounding
def test_philox_known_answers():
    """Both oracles' Philox4x32-10 against the published known-answer vectors (tests/golden/philox4x32_10_kat.txt)."""
    import os
    rows = [ln.split() for ln in open(os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        ctr, key, want = w[0:4], w[4:6], w[6:10]
        assert npo.philox4x32_10(np.array(ctr), np.array(key)).tolist() == want
        assert co.philox4x32_10(ctr, key).tolist() == want
    # vectorised over many counters = one at a time
    rng = np.random.RandomState(31)
    ctrs = rng.randint(0, 2 ** 32, size=(50, 4), dtype=np.uint64)
    key = rng.randint(0, 2 ** 32, size=2, dtype=np.uint64)
    many = npo.philox4x32_10(ctrs, key)
    for c, o in zip(ctrs, many):
        assert co.philox4x32_10(c, key).tolist() == o.tolist()


def test_stochastic_rounding_is_exactly_unbiased_and_leaves_bf16_values_alone():
    """Closed form: over all 65536 values of the random integer, a float x between the bfloat16 neighbours a < b (in
    magnitude) goes to b exactly low16(x) times, so the mean of the results is x itself; a bfloat16 value never moves."""
    rng = np.random.RandomState(32)
    xs = np.concatenate([(rng.standard_normal(40) * 10.0 ** rng.uniform(-30, 30, 40)).astype(np.float32),
                         np.array([1.0, -1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -23, 2.0 - 2.0 ** -23, 1e-40, -3e-39], np.float32)])
    r = np.arange(65536, dtype=np.uint32)
    for x in xs:
        out = npo.stochastic_round_to_bf16(np.full(65536, x, np.float32), r).astype(np.float64)
        lo16 = int(np.float32(x).view(np.uint32)) & 0xFFFF
        vals = np.unique(out)
        assert len(vals) == (1 if lo16 == 0 else 2)
        assert (out.astype(np.float32).view(np.uint32) & 0xFFFF == 0).all()
        assert int((np.abs(out) == np.abs(vals).max()).sum()) == (65536 if lo16 == 0 else lo16)
        assert abs(out.mean() - float(x)) <= 2.0 ** -40 * abs(float(x))            # = x up to the float64 mean's rounding
    # C and numpy agree, value by value; infinities and NaN are rounded to nearest
    for x, rr in zip(xs, rng.randint(0, 65536, size=len(xs))):
        want = int(npo.stochastic_round_to_bf16(np.array([x], np.float32), np.array([rr]))[0].view(np.uint32)) >> 16
        assert co.float_to_bf16_stochastic_bits(x, int(rr)) == want
    assert co.float_to_bf16_stochastic_bits(np.inf, 65535) == 0x7F80 and co.float_to_bf16_stochastic_bits(-np.inf, 1) == 0xFF80
    assert np.isinf(npo.stochastic_round_to_bf16(np.array([np.inf], np.float32), np.array([65535]))[0])


def test_stochastic_step_is_the_nearest_rounding_steps_value_rounded_with_the_stated_random_numbers():
    """The C oracle's stochastic step, piece by piece: its single-precision m' and v' are those of the (exact-arithmetic
    pinned) fp32-decision mode -- recovered here as the values whose two candidate roundings bracket them -- and the
    stored result is stochastic_round_to_bf16 of that value with rounding_randoms(arena position, step, seed)."""
    rng = np.random.RandomState(33)
    n, index0, step, seed = 5000, 123456, 7, 0x1234_5678_9ABC_DEF0
    g = bf16_values(rng, n, 1e-4).astype(np.float32)
    m0, v0 = bf16_values(rng, n, 3e-5), np.abs(bf16_values(rng, n, 1e-8))
    theta = (rng.standard_normal(n) * 0.02).astype(np.float32)
    # the single-precision values, by the numpy route: products of two floats are exact in float64, and the one
    # float64 addition is exact whenever both terms fit 53 bits together, which holds for all but a few elements
    h, b1, b2 = np.float32(0.61), np.float32(0.9), np.float32(0.95)
    o1, o2 = np.float32(1.0 - 0.9), np.float32(1.0 - 0.95)
    gh = (h * g).astype(np.float32)
    m1f = (b1.astype(np.float64) * m0.astype(np.float64) + (o1 * gh).astype(np.float32).astype(np.float64)).astype(np.float32)
    v1f = (b2.astype(np.float64) * v0.astype(np.float64) +
           (o2 * (gh * gh).astype(np.float32)).astype(np.float32).astype(np.float64)).astype(np.float32)
    idx = index0 + np.arange(n)
    rm, rv = npo.rounding_randoms(idx, step, seed)
    want_m = (npo.stochastic_round_to_bf16(m1f, rm).view(np.uint32) >> 16).astype(np.uint16)
    want_v = (npo.stochastic_round_to_bf16(v1f, rv).view(np.uint32) >> 16).astype(np.uint16)
    th_s, mb, vb = theta.copy(), f32_to_bits(m0), f32_to_bits(v0)
    co.adamw_update_bf16state(th_s, g, mb, vb, float(h), step, 3e-4, 0.9, 0.95, 1e-8, 0.1, fp32_decision=True,
                              stochastic_seed=seed, index0=index0)
    assert (mb != want_m).mean() < 1e-3 and (vb != want_v).mean() < 1e-3          # (double rounding of the numpy route)
    assert (np.abs(mb.astype(np.int64) - want_m.astype(np.int64)) <= 1).all()
    # an explicit index array gives the same as index0 + j, another step or seed gives other roundings, theta is untouched
    th2, mb2, vb2 = theta.copy(), f32_to_bits(m0), f32_to_bits(v0)
    co.adamw_update_bf16state(th2, g, mb2, vb2, float(h), step, 3e-4, 0.9, 0.95, 1e-8, 0.1, fp32_decision=True,
                              stochastic_seed=seed, index=idx.astype(np.int64))
    assert np.array_equal(mb, mb2) and np.array_equal(vb, vb2) and np.array_equal(th_s, th2)
    th3, mb3, vb3 = theta.copy(), f32_to_bits(m0), f32_to_bits(v0)
    co.adamw_update_bf16state(th3, g, mb3, vb3, float(h), step, 3e-4, 0.9, 0.95, 1e-8, 0.1, fp32_decision=True)
    assert np.array_equal(th3, th_s)                                           # theta never sees the rounding
    assert 0.2 < (mb3 != mb).mean() < 0.3        # a uniform fraction f goes the other way with probability min(f, 1 - f): 1/4
    # stochastic and nearest results are the two neighbours of the same value
    assert (np.abs(mb3.astype(np.int64) - mb.astype(np.int64)) <= 1).all()
    th4, mb4, vb4 = theta.copy(), f32_to_bits(m0), f32_to_bits(v0)
    co.adamw_update_bf16state(th4, g, mb4, vb4, float(h), step + 1, 3e-4, 0.9, 0.95, 1e-8, 0.1, fp32_decision=True,
                              stochastic_seed=seed, index0=index0)
    assert (mb4 != mb).mean() > 0.2


def test_stochastic_rounding_tracks_a_slow_average_where_nearest_rounding_stalls():
    """Why one would round stochastically: with beta2 = 0.999 a bfloat16 v rounded to nearest stops moving 500 spacings
    (a factor of several) short of its fixed point, while the stochastically rounded v reaches it on average."""
    n = 4096
    g = np.full(n, 1e-3, np.float32)
    theta = np.zeros(n, np.float32)
    res = {}
    for mode, seed in (("nearest", None), ("stochastic", 99)):
        th, mb, vb = theta.copy(), np.zeros(n, np.uint16), np.zeros(n, np.uint16)
        for t in range(1, 6001):
            co.adamw_update_bf16state(th, g, mb, vb, 1.0, t, 0.0, 0.9, 0.999, 1e-8, 0.0, fp32_decision=True,
                                      stochastic_seed=seed)
        res[mode] = bits_to_f64(vb)
    target = 1e-6 * (1 - 0.999 ** 6000)
    assert res["nearest"].max() < 0.5 * target                                  # stalled far below
    assert abs(res["stochastic"].mean() - target) < 0.02 * target               # unbiased
    assert res["stochastic"].std() < 0.1 * target
