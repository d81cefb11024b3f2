"""CPU oracle for AdamW with AdaGC (Algorithm 1 of the paper; Eq. 2 and Eq. 3).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, float64 restatement of the
paper's algorithm used to check the CUDA library.  It shares no code with the
CUDA path and is never a fallback for it: only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it.

Every function takes the steps of Algorithm 1 in the paper's order and notation:

    g_t,i      gradient of tensor i at step t (t is 1-based: the first call is t = 1)
    gamma_i    EMA of the clipped gradient norm of tensor i (one fp32 per tensor,
               Section 4.3 "Memory")
    h_t,i      clip factor, hat(g) = h * g
    m, v       AdamW moments, theta the parameters

Readings taken where the paper is silent or ambiguous (listed in the design notes):
  * warm-up covers exactly T_start steps: steps 1..T_start use global-norm
    clipping (Eq. 2), step T_start+1 is the first per-tensor AdaGC step (Eq. 3);
  * the warm-up EMA seed uses the globally *clipped* per-tensor norm
    (Algorithm 1 writes the hatted gradient there);
  * at t = 1 the incoming gamma is ignored: gamma_0,i = ||hat(g)_1,i||;
    with T_start = 0 the first step seeds gamma_0,i = ||g_1,i|| and then applies Eq. 3;
  * the clip is active only when ||g|| > lambda_rel * gamma (strict), and the
    clipped norm that enters the EMA is then lambda_rel * gamma itself
    (Section 4.2: the clip "scales the gradient norm to" that value);
  * stored state (gamma, theta, m, v) is rounded to its storage dtype after every
    step ("storage" mode, the parity reference); `state_dtype=np.float64` keeps
    everything in float64 for invariant tests;
  * with `moment_dtype="bf16"` the moments are STORED as bfloat16 (the paper trains in
    bfloat16 / float8 precision and does not say how optimizer state is rounded): a step reads
    the stored bfloat16 moments exactly, does its arithmetic in float64, updates theta from
    the unrounded new moments, and rounds the moments to the nearest bfloat16 (ties to even)
    only when it stores them.

Parity pins: tests/test_oracle_pins.py (closed forms, library special cases,
hand-worked example, invariants, brute force).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np


@dataclass
class Hyper:
    """The 'given' line of Algorithm 1 (eta_t is passed per step as `lr`)."""
    lr: float = 3e-4
    beta1: float = 0.9
    beta2: float = 0.95
    eps: float = 1e-8
    wd: float = 0.1          # lambda_w
    lambda_rel: float = 1.04
    beta: float = 0.99
    lambda_abs: float = 1.0
    warmup: int = 100        # T_start


@dataclass
class ClipResult:
    norm: np.ndarray      # ||g_t,i||                       float64 [T]
    h: np.ndarray         # clip factor h_t,i               float64 [T]
    flag: np.ndarray      # clip active                     bool    [T]
    clipped: np.ndarray   # ||hat(g)_t,i||                  float64 [T]
    gamma: np.ndarray     # gamma_t,i in the state dtype    [T]
    global_norm: float    # ||g_t|| (Eq. 2), always reported
    margin: np.ndarray    # |norm - threshold| / threshold of every decision (inf where threshold is 0)


def sumsq(g: np.ndarray) -> float:
    """sum_j g_j^2 of one tensor in float64 (the square of the norm in Eq. 3)."""
    x = np.asarray(g, dtype=np.float64).ravel()
    return float(np.sum(x * x))


def l2_norm(g: np.ndarray) -> float:
    return math.sqrt(sumsq(g))


def _bf16_grid(x: np.ndarray):
    """For finite non-zero float64 x: (q, p) with x = q * 2^(p-7), where 2^(p-7) is the spacing of bfloat16
    values around x.  bfloat16 has 8 significand bits (one implicit, seven stored), the exponent range of
    float32 (normal numbers from 2^-126) and subnormals with the fixed spacing 2^-133 below that."""
    _, e = np.frexp(x)                                   # |x| = frac * 2^e with frac in [0.5, 1)
    p = np.maximum(e - 1, -126)                          # floor(log2|x|), clamped for subnormals
    return np.ldexp(x, 7 - p), p


def round_to_bf16(x) -> np.ndarray:
    """Nearest bfloat16 value of every element (round to nearest, ties to even), returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    y = x.copy()
    fin = np.isfinite(x) & (x != 0.0)
    q, p = _bf16_grid(x[fin])
    r = np.ldexp(np.rint(q), p - 7)                      # np.rint rounds halves to even
    r[np.abs(r) >= 2.0 ** 128] = np.inf * np.sign(r[np.abs(r) >= 2.0 ** 128])    # beyond the largest finite value
    y[fin] = r
    return y


def bf16_rounding_margin(x, scale) -> np.ndarray:
    """How far each x is from the nearest point where rounding to bfloat16 changes its result (the midpoint
    between two neighbouring bfloat16 values), divided by `scale`.  An implementation whose x differs from
    this oracle's by less than margin * scale rounds to the same bfloat16."""
    x = np.asarray(x, dtype=np.float64)
    out = np.full(x.shape, np.inf)
    fin = np.isfinite(x) & (x != 0.0)
    q, p = _bf16_grid(x[fin])
    frac = np.abs(q) - np.floor(np.abs(q))
    dist = np.abs(frac - 0.5)                            # in units of the spacing 2^(p-7)
    # just above a power of two the values below are twice as dense: the flip below 2^p is a quarter spacing under it
    low_edge = (np.floor(np.abs(q)) == 128.0) & (p > -126)
    dist = np.where(low_edge, np.minimum(dist, frac + 0.25), dist)
    with np.errstate(divide="ignore", invalid="ignore"):
        out[fin] = dist * np.ldexp(1.0, p - 7) / np.broadcast_to(np.asarray(scale, np.float64), x.shape)[fin]
    return out


# ----------------------------------------------------------------------------------------------------------------
# Stochastic rounding of stored bfloat16 moments.  The random numbers come from the counter-based generator
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011), written here from
# its definition: a counter of four 32-bit words and a key of two go through ten rounds; a round replaces the counter
# (c0, c1, c2, c3) by (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)), where hi / lo are the halves
# of the 64-bit product, and after each round but the last the key is bumped by the Weyl constants (W0, W1).
# ----------------------------------------------------------------------------------------------------------------
PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter, key) -> np.ndarray:
    """counter: (..., 4) uint32 words, key: (2,) or (..., 2) uint32 words -> (..., 4) uint32 output words."""
    c = np.asarray(counter, dtype=np.uint64) & 0xFFFFFFFF
    k = np.broadcast_to(np.asarray(key, dtype=np.uint64) & 0xFFFFFFFF, c.shape[:-1] + (2,))
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = k[..., 0].copy(), k[..., 1].copy()
    mask = np.uint64(0xFFFFFFFF)
    for r in range(10):
        p0, p1 = np.uint64(PHILOX_M0) * c0, np.uint64(PHILOX_M1) * c2          # 32 x 32 -> 64 bits, exact in uint64
        c0, c1, c2, c3 = (p1 >> np.uint64(32)) ^ c1 ^ k0, p1 & mask, (p0 >> np.uint64(32)) ^ c3 ^ k1, p0 & mask
        if r < 9:
            k0, k1 = (k0 + np.uint64(PHILOX_W0)) & mask, (k1 + np.uint64(PHILOX_W1)) & mask
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def rounding_randoms(index: np.ndarray, step: int, seed: int):
    """The two 16-bit random numbers (for m and for v) of the elements at arena positions `index` at step `step`:
    the group of four elements 4q..4q+3 shares one generator call with counter (lo(q), hi(q), lo(step), hi(step)) and
    key (lo(seed), hi(seed)); element 4q + l takes output word l, its low half for m and its high half for v."""
    index = np.asarray(index, dtype=np.uint64)
    q = index >> np.uint64(2)
    ctr = np.stack([q & np.uint64(0xFFFFFFFF), q >> np.uint64(32),
                    np.full(q.shape, step & 0xFFFFFFFF, np.uint64), np.full(q.shape, (step >> 32) & 0xFFFFFFFF, np.uint64)], axis=-1)
    out = philox4x32_10(ctr, np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], np.uint64))
    word = np.take_along_axis(out, (index & np.uint64(3)).astype(np.int64)[..., None], axis=-1)[..., 0]
    return (word & np.uint32(0xFFFF)).astype(np.uint32), (word >> np.uint32(16)).astype(np.uint32)


def stochastic_round_to_bf16(x32: np.ndarray, r16: np.ndarray) -> np.ndarray:
    """Stochastic rounding of float32 values to bfloat16 with the 16-bit random integers r16: the value moves to the
    neighbour of larger magnitude with probability (distance to the smaller neighbour) / spacing, which is what adding
    r16 to the low half of the float32 bit pattern and dropping that half does (a carry runs into the exponent as it
    should); bfloat16 values are left as they are, infinities and NaN are rounded to nearest.  Returns the bfloat16
    values held in float32."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    u = x32.view(np.uint32).astype(np.uint64)
    out = (((u + np.asarray(r16, np.uint64)) >> np.uint64(16)) << np.uint64(16)).astype(np.uint32).view(np.float32)
    special = ~np.isfinite(x32)
    if special.any():
        out = out.copy()
        out[special] = round_to_bf16(x32[special].astype(np.float64)).astype(np.float32)
    return out


def clip_decisions(s: Sequence[float], gamma_prev: np.ndarray, step: int, hp: Hyper,
                   state_dtype=np.float32, keep_initial: bool = False,
                   global_adaptive: bool = False, ema_cap: Optional[float] = None) -> ClipResult:
    """Clip factors, flags and the EMA update for one step, from per-tensor sums of squares.

    Warm-up branch: Eq. 2 and the min-seeding line of Algorithm 1.
    AdaGC branch:   Eq. 3 and the gamma update of Algorithm 1.

    Two variants of the paper's ablations (Section 5, "EMA Initialization Strategy" and "Adaptivity Efficacy
    and Locality Granularity"):
      keep_initial    gamma is not seeded at t = 1; the caller's gamma_0 (e.g. the constant 0.5 or 1.0 of
                      the ablation) is used as gamma_{t-1} from the first step on;
      global_adaptive "Global AdaGC": one adaptive threshold for the whole model, i.e. this same algorithm
                      applied to the single tensor that all gradients form together; every tensor gets
                      that one clip factor, flag and gamma;
      ema_cap         "thresholded initialization" (variant 3 of the EMA-initialization ablation, cap 0.1 there):
                      gamma_t,i = min(||hat(g)_t,i||, ema_cap) wherever the default seeds gamma or takes the
                      running minimum; the constant stands where gamma_t-1,i stood, so no warm-up step
                      remembers the one before it.
    """
    if global_adaptive:
        s_all = np.asarray(s, dtype=np.float64)
        one = clip_decisions([float(np.sum(s_all))], np.asarray(gamma_prev)[:1], step, hp, state_dtype,
                             keep_initial, False, ema_cap)
        T = s_all.shape[0]
        n_i = np.sqrt(s_all)
        return ClipResult(n_i, np.full(T, one.h[0]), np.full(T, bool(one.flag[0])), one.h[0] * n_i,
                          np.full(T, one.gamma[0], dtype=state_dtype), one.global_norm,
                          np.full(T, one.margin[0]))
    seed = step == 1 and not keep_initial
    s = np.asarray(s, dtype=np.float64)
    T = s.shape[0]
    n = np.sqrt(s)                                         # ||g_t,i||
    G = math.sqrt(float(np.sum(s)))                        # ||g_t|| over all tensors
    h = np.ones(T, dtype=np.float64)
    flag = np.zeros(T, dtype=bool)
    c = np.empty(T, dtype=np.float64)
    margin = np.full(T, np.inf)
    gam = np.asarray(gamma_prev).astype(state_dtype).astype(np.float64)
    if step < 1:
        raise ValueError("step is 1-based")

    if step <= hp.warmup:
        # h_t = min{lambda_abs / ||g_t||, 1}
        clip_all = G > hp.lambda_abs
        h_t = hp.lambda_abs / G if clip_all else 1.0
        if hp.lambda_abs > 0:
            margin[:] = abs(G - hp.lambda_abs) / hp.lambda_abs
        for i in range(T):
            h[i] = h_t
            flag[i] = clip_all
            c[i] = h_t * n[i]                              # ||hat(g)_t,i||
            # gamma_t,i = min{gamma_t-1,i, ||hat(g)_t,i||},  gamma_0,i = ||hat(g)_1,i||
            if ema_cap is not None and ema_cap > 0:
                gam[i] = c[i] if c[i] < ema_cap else ema_cap
            else:
                gam[i] = c[i] if seed else min(gam[i], c[i])
    else:
        for i in range(T):
            if seed:                                       # T_start = 0: seed, then Eq. 3
                gam[i] = float(np.asarray(n[i]).astype(state_dtype))
                if ema_cap is not None and ema_cap > 0 and not gam[i] < ema_cap:
                    gam[i] = ema_cap
            thr = hp.lambda_rel * gam[i]
            if thr > 0:
                margin[i] = abs(n[i] - thr) / thr
            if n[i] > thr:                                 # clip active
                flag[i] = True
                h[i] = thr / n[i]                          # lambda_rel * gamma / ||g||
                c[i] = thr                                 # norm scaled to lambda_rel * gamma
            else:
                h[i] = 1.0
                c[i] = n[i]
            # gamma_t,i = beta * gamma_t-1,i + (1 - beta) * ||hat(g)_t,i||
            gam[i] = hp.beta * gam[i] + (1.0 - hp.beta) * c[i]
    return ClipResult(n, h, flag, c, gam.astype(state_dtype), G, margin)


def adamw_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, h: float,
                 step: int, hp: Hyper, state_dtype=np.float32, moment_dtype: Optional[str] = None,
                 return_margin: bool = False):
    """The four AdamW lines of Algorithm 1 on hat(g) = h * g, elementwise, in float64.

    Inputs are read in their storage dtype, the arithmetic is float64, the results are
    rounded to `state_dtype`.  Works on any array of elements of one tensor (or a sample).

    moment_dtype="bf16": m and v are stored as bfloat16 (held here in float32 arrays whose values are
    bfloat16 values).  theta is updated from the unrounded new moments; the moments are rounded to the
    nearest bfloat16, ties to even, when stored.  Rounding is a discrete decision: with `return_margin`
    the call also returns, per element, how close m and v came to a point where the rounding flips,
    relative to the size of the terms they are summed from (see bf16_rounding_margin).
    """
    th = np.asarray(theta, dtype=np.float64)
    gh = float(h) * np.asarray(g, dtype=np.float64)                   # hat(g)
    m1 = hp.beta1 * np.asarray(m, dtype=np.float64) + (1.0 - hp.beta1) * gh
    v1 = hp.beta2 * np.asarray(v, dtype=np.float64) + (1.0 - hp.beta2) * gh * gh
    m_hat = m1 / (1.0 - hp.beta1 ** step)
    v_hat = v1 / (1.0 - hp.beta2 ** step)
    th1 = th - hp.lr * hp.wd * th - hp.lr * m_hat / (np.sqrt(v_hat) + hp.eps)
    if moment_dtype is None:
        return th1.astype(state_dtype), m1.astype(state_dtype), v1.astype(state_dtype)
    if moment_dtype != "bf16":
        raise ValueError("moment_dtype is None or 'bf16'")
    out = (th1.astype(state_dtype), round_to_bf16(m1).astype(np.float32), round_to_bf16(v1).astype(np.float32))
    if return_margin:
        old_term = hp.beta1 * np.asarray(m, dtype=np.float64)      # m1 = old_term + (m1 - old_term): its two terms
        m_scale = np.abs(old_term) + np.abs(m1 - old_term)
        return out + (bf16_rounding_margin(m1, m_scale), bf16_rounding_margin(v1, np.abs(v1)))
    return out


def lion_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, h: float, lr: float, beta1: float,
                beta2: float, wd: float, state_dtype=np.float32, return_margin: bool = False,
                moment_dtype: Optional[str] = None):
    """Lion on the clipped gradient hat(g) = h * g (Section 4.2 of the paper: the clip is
    optimizer-agnostic and is used with Lion; the update itself is Lion's published rule,
    Chen et al. 2023):
        c     = beta1 * m + (1 - beta1) * hat(g)
        theta = theta - lr * (sign(c) + wd * theta)        (decoupled decay on theta_{t-1})
        m     = beta2 * m + (1 - beta2) * hat(g)
    Elementwise, float64 arithmetic, results rounded to `state_dtype`.

    sign(c) is a discrete decision.  Where the two terms of c nearly cancel, an implementation that
    rounds differently (float32 arithmetic, a stored m that differs in its last bit) may legitimately
    take the other sign; with `return_margin` the relative margin |c| / (|beta1 m| + |(1-beta1) hat(g)|)
    of every element is returned too, so that a comparison can tell such near-ties from real errors."""
    th = np.asarray(theta, dtype=np.float64)
    mm = np.asarray(m, dtype=np.float64)
    gh = float(h) * np.asarray(g, dtype=np.float64)
    a, b = beta1 * mm, (1.0 - beta1) * gh
    c = a + b
    th1 = th - lr * (np.sign(c) + wd * th)
    m1 = beta2 * mm + (1.0 - beta2) * gh
    # moment_dtype="bf16": the momentum is stored as bfloat16, rounded to nearest even on store
    out = (th1.astype(state_dtype), m1.astype(state_dtype) if moment_dtype is None else round_to_bf16(m1).astype(np.float32))
    if return_margin:
        den = np.abs(a) + np.abs(b)
        with np.errstate(divide="ignore", invalid="ignore"):
            margin = np.where(den > 0, np.abs(c) / den, np.inf)
        return out + (margin,)
    return out


def sgdm_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, h: float, lr: float, momentum: float,
                wd: float, state_dtype=np.float32, moment_dtype: Optional[str] = None) -> Tuple[np.ndarray, np.ndarray]:
    """SGD with momentum on the clipped gradient hat(g) = h * g (Section 4.2: the clip is optimizer-agnostic).
    The textbook heavy-ball form with L2 weight decay folded into the gradient, the form common libraries use:
        d     = hat(g) + wd * theta
        m     = momentum * m + d              (m_0 = 0)
        theta = theta - lr * m
    Elementwise, float64 arithmetic, results rounded to `state_dtype`."""
    th = np.asarray(theta, dtype=np.float64)
    d = float(h) * np.asarray(g, dtype=np.float64) + wd * th
    m1 = momentum * np.asarray(m, dtype=np.float64) + d
    th1 = th - lr * m1                                    # theta sees the unrounded momentum
    return th1.astype(state_dtype), m1.astype(state_dtype) if moment_dtype is None else round_to_bf16(m1).astype(np.float32)


def clipped_grad(g: np.ndarray, h: float) -> np.ndarray:
    """hat(g) = h * g in float64 (the clip-only use of the method with other optimizers)."""
    return float(h) * np.asarray(g, dtype=np.float64)


class AdaGCAdamW:
    """Algorithm 1 over a list of tensors; holds theta, m, v, gamma and the counters."""

    def __init__(self, params: Sequence[np.ndarray], hp: Hyper, state_dtype=np.float32,
                 moment_dtype: Optional[str] = None):
        self.hp = hp
        self.dt = state_dtype
        self.moment_dtype = moment_dtype
        self.theta = [np.array(p, dtype=state_dtype) for p in params]
        self.m = [np.zeros_like(p) for p in self.theta]               # m_0 = 0
        self.v = [np.zeros_like(p) for p in self.theta]               # v_0 = 0
        self.gamma = np.zeros(len(self.theta), dtype=state_dtype)
        self.t = 0
        self.clip_count = np.zeros(len(self.theta), dtype=np.uint64)
        self.last: Optional[ClipResult] = None

    def clip(self, grads: Sequence[np.ndarray]) -> ClipResult:
        """The clipping half of one step: advances t, gamma and the counters."""
        self.t += 1
        s = [sumsq(g) for g in grads]
        r = clip_decisions(s, self.gamma, self.t, self.hp, self.dt)
        self.gamma = r.gamma
        self.clip_count += r.flag.astype(np.uint64)
        self.last = r
        return r

    def step(self, grads: Sequence[np.ndarray], lr: Optional[float] = None) -> ClipResult:
        r = self.clip(grads)
        hp = self.hp if lr is None else Hyper(**{**self.hp.__dict__, "lr": lr})
        for i, g in enumerate(grads):
            self.theta[i], self.m[i], self.v[i] = adamw_update(
                self.theta[i], g, self.m[i], self.v[i], r.h[i], self.t, hp, self.dt, self.moment_dtype)
        return r

    def clip_only(self, grads: Sequence[np.ndarray]) -> Tuple[ClipResult, List[np.ndarray]]:
        r = self.clip(grads)
        return r, [clipped_grad(g, r.h[i]) for i, g in enumerate(grads)]
