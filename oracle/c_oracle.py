"""ctypes front end of the C oracle (adagc_ref.c).  TEST INFRASTRUCTURE ONLY.

Same role as adagc_oracle.py (Algorithm 1, Eq. 2, Eq. 3 of the paper in float64), but fast
enough for layouts with 1e8..1e10 elements.  bf16 gradients are passed as uint16 arrays of
their bit patterns.  Never imported by the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adagc_ref.c")
_LIB = os.path.join(_HERE, "libadagc_ref.so")
_lib = None

_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(np.int64, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")


def build(force: bool = False) -> str:
    """Compile adagc_ref.c into libadagc_ref.so next to it (gcc, OpenMP, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.adagc_ref_num_threads.restype = C.c_int
        L.adagc_ref_double_to_bf16.restype = C.c_uint16
        L.adagc_ref_double_to_bf16.argtypes = [C.c_double]
        L.adagc_ref_sumsq.restype = C.c_double
        L.adagc_ref_sumsq.argtypes = [C.c_void_p, C.c_int, C.c_int64]
        L.adagc_ref_sumsq_tensors.restype = None
        L.adagc_ref_sumsq_tensors.argtypes = [C.c_void_p, C.c_int, C.c_int32, _i64p, _i64p, _f64p]
        L.adagc_ref_clip_decisions.restype = None
        L.adagc_ref_clip_decisions.argtypes = [C.c_int32, _f64p, _f32p, C.c_int64, C.c_double, C.c_double,
                                               C.c_double, C.c_int64, _f64p, _f64p, _u8p, _f64p, _f64p, _f64p]
        L.adagc_ref_clip_decisions_ex.restype = None
        L.adagc_ref_clip_decisions_ex.argtypes = [C.c_int32, _f64p, _f32p, C.c_int64, C.c_double, C.c_double,
                                                  C.c_double, C.c_int64, C.c_int, _f64p, _f64p, _u8p, _f64p, _f64p,
                                                  _f64p]
        L.adagc_ref_clip_decisions_cap.restype = None
        L.adagc_ref_clip_decisions_cap.argtypes = [C.c_int32, _f64p, _f32p, C.c_int64, C.c_double, C.c_double,
                                                   C.c_double, C.c_int64, C.c_int, C.c_double, _f64p, _f64p, _u8p,
                                                   _f64p, _f64p, _f64p]
        L.adagc_ref_adamw.restype = None
        L.adagc_ref_adamw.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64,
                                      C.c_double, C.c_int64] + [C.c_double] * 5
        L.adagc_ref_lion.restype = None
        L.adagc_ref_lion.argtypes = ([C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int64] + [C.c_double] * 5 +
                                     [C.c_void_p, C.c_double])
        L.adagc_ref_sgdm.restype = None
        L.adagc_ref_sgdm.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int64] + [C.c_double] * 4
        L.adagc_ref_adamw_bf16state.restype = None
        L.adagc_ref_adamw_bf16state.argtypes = ([C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64,
                                                 C.c_double, C.c_int64] + [C.c_double] * 5 +
                                                [C.c_void_p, C.c_double, C.c_int, C.c_int, C.c_uint64, C.c_int64,
                                                 C.c_void_p])
        L.adagc_ref_lion_bf16state.restype = None
        L.adagc_ref_lion_bf16state.argtypes = ([C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int64] +
                                               [C.c_double] * 5 + [C.c_void_p, C.c_double, C.c_int, C.c_int,
                                                                   C.c_uint64, C.c_int64, C.c_int64])
        L.adagc_ref_sgdm_bf16state.restype = None
        L.adagc_ref_sgdm_bf16state.argtypes = ([C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int64] +
                                               [C.c_double] * 4 + [C.c_void_p, C.c_double, C.c_int, C.c_int,
                                                                   C.c_uint64, C.c_int64, C.c_int64])
        L.adagc_ref_philox4x32_10.restype = None
        L.adagc_ref_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.adagc_ref_float_to_bf16_stochastic.restype = C.c_uint16
        L.adagc_ref_float_to_bf16_stochastic.argtypes = [C.c_float, C.c_uint32]
        L.adagc_ref_scale.restype = None
        L.adagc_ref_scale.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_double]
        L.adagc_ref_step.restype = C.c_int32
        L.adagc_ref_step.argtypes = ([C.c_int32, _i64p, _i64p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                      C.c_void_p, _f32p, C.c_int64] + [C.c_double] * 8 + [C.c_int64] +
                                     [_f64p, _f64p, _f64p, _u8p, _f64p, _f64p, _f64p])
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().adagc_ref_num_threads())


def _grad_ptr(g: np.ndarray) -> Tuple[int, int]:
    assert g.flags["C_CONTIGUOUS"]
    if g.dtype == np.uint16:
        return g.ctypes.data, 1
    if g.dtype == np.float32:
        return g.ctypes.data, 0
    raise TypeError("gradients must be float32, or uint16 holding bf16 bit patterns")


def sumsq(g: np.ndarray) -> float:
    p, bf = _grad_ptr(g)
    return float(lib().adagc_ref_sumsq(p, bf, g.size))


def sumsq_tensors(arena: np.ndarray, offsets: Sequence[int], numels: Sequence[int]) -> np.ndarray:
    p, bf = _grad_ptr(arena)
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    nel = np.ascontiguousarray(numels, dtype=np.int64)
    out = np.empty(len(off), dtype=np.float64)
    lib().adagc_ref_sumsq_tensors(p, bf, len(off), off, nel, out)
    return out


def clip_decisions(s: np.ndarray, gamma: np.ndarray, step: int, lambda_rel: float, beta: float,
                   lambda_abs: float, warmup: int, keep_initial: bool = False, global_adaptive: bool = False,
                   ema_cap: float = 0.0):
    """Returns dict(norm, h, flag, clipped, margin, global_norm); `gamma` (fp32) is updated in place.
    ema_cap > 0 selects the "thresholded initialization" variant (gamma = min(clipped norm, ema_cap) in warm-up)."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    T = len(s)
    assert gamma.dtype == np.float32 and gamma.flags["C_CONTIGUOUS"] and len(gamma) == T
    norm, h, clipped, margin = (np.empty(T, np.float64) for _ in range(4))
    flag = np.empty(T, np.uint8)
    G = np.empty(1, np.float64)
    variant = (1 if keep_initial else 0) | (2 if global_adaptive else 0)
    lib().adagc_ref_clip_decisions_cap(T, s, gamma, step, lambda_rel, beta, lambda_abs, warmup, variant,
                                       float(ema_cap), norm, h, flag, clipped, margin, G)
    return dict(norm=norm, h=h, flag=flag.astype(bool), clipped=clipped, margin=margin,
                global_norm=float(G[0]), gamma=gamma)


def adamw_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, h: float, step: int,
                 lr: float, beta1: float, beta2: float, eps: float, wd: float) -> None:
    """In place on fp32 theta, m, v."""
    p, bf = _grad_ptr(g)
    for a in (theta, m, v):
        assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"] and a.size == g.size
    lib().adagc_ref_adamw(theta.ctypes.data, p, bf, m.ctypes.data, v.ctypes.data, g.size,
                          float(h), int(step), lr, beta1, beta2, eps, wd)


def _tie_ptr(near_tie: Optional[np.ndarray], n: int):
    if near_tie is None:
        return None
    assert near_tie.dtype == np.uint8 and near_tie.flags["C_CONTIGUOUS"] and near_tie.size == n
    return near_tie.ctypes.data


def _is_bf16_state(theta: np.ndarray, moments, n: int) -> bool:
    """Moments are fp32 arrays, or uint16 arrays holding bfloat16 bit patterns (all of one kind)."""
    assert theta.dtype == np.float32 and theta.flags["C_CONTIGUOUS"] and theta.size == n
    kinds = {a.dtype for a in moments}
    assert kinds in ({np.dtype(np.float32)}, {np.dtype(np.uint16)}), "moments: all float32, or all uint16 (bf16 bits)"
    for a in moments:
        assert a.flags["C_CONTIGUOUS"] and a.size == n
    return kinds == {np.dtype(np.uint16)}


def adamw_update_bf16state(theta: np.ndarray, g: np.ndarray, m: np.ndarray, v: np.ndarray, h: float, step: int,
                           lr: float, beta1: float, beta2: float, eps: float, wd: float,
                           near_tie: Optional[np.ndarray] = None, tie_tol: float = 0.0,
                           fp32_decision: bool = False, stochastic_seed: Optional[int] = None, index0: int = 0,
                           index: Optional[np.ndarray] = None) -> None:
    """AdamW with m and v stored as bfloat16 (uint16 bit patterns), in place; theta fp32.  `near_tie` (uint8) counts,
    per element, the steps in which the float64 rounding of m or v was decided with a relative margin below `tie_tol`.
    fp32_decision: the value rounded to bfloat16 is evaluated in single precision (see adagc_ref.c) instead.
    stochastic_seed: round that value stochastically, with the random numbers of the elements' arena positions
    (`index`, an int64 array, or index0 + j), the step and this seed."""
    p, bf = _grad_ptr(g)
    assert _is_bf16_state(theta, (m, v), g.size)
    assert stochastic_seed is None or fp32_decision, "stochastic rounding acts on the single-precision value"
    if index is not None:
        assert index.dtype == np.int64 and index.flags["C_CONTIGUOUS"] and index.size == g.size
    lib().adagc_ref_adamw_bf16state(theta.ctypes.data, p, bf, m.ctypes.data, v.ctypes.data, g.size, float(h),
                                    int(step), lr, beta1, beta2, eps, wd, _tie_ptr(near_tie, g.size), float(tie_tol),
                                    int(fp32_decision), int(stochastic_seed is not None), int(stochastic_seed or 0),
                                    int(index0), None if index is None else index.ctypes.data)


def lion_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, h: float, lr: float, beta1: float,
                beta2: float, wd: float, near_tie: Optional[np.ndarray] = None, tie_tol: float = 0.0,
                fp32_decision: bool = False, stochastic_seed: Optional[int] = None, step: int = 0,
                index0: int = 0) -> None:
    """Lion on the clipped gradient, in place on fp32 theta and on m (fp32, or uint16 = stored as bfloat16).
    `near_tie` (uint8, same length) counts, per element, the steps in which sign(c) -- and, for bfloat16 m, its
    rounding -- was decided with a relative margin below `tie_tol`."""
    p, bf = _grad_ptr(g)
    nt = _tie_ptr(near_tie, g.size)
    if _is_bf16_state(theta, (m,), g.size):
        lib().adagc_ref_lion_bf16state(theta.ctypes.data, p, bf, m.ctypes.data, g.size, float(h), lr, beta1, beta2,
                                       wd, nt, float(tie_tol), int(fp32_decision), int(stochastic_seed is not None),
                                       int(stochastic_seed or 0), int(step), int(index0))
    else:
        lib().adagc_ref_lion(theta.ctypes.data, p, bf, m.ctypes.data, g.size, float(h), lr, beta1, beta2, wd,
                             nt, float(tie_tol))


def sgdm_update(theta: np.ndarray, g: np.ndarray, m: np.ndarray, h: float, lr: float, momentum: float,
                wd: float, near_tie: Optional[np.ndarray] = None, tie_tol: float = 0.0,
                fp32_decision: bool = False, stochastic_seed: Optional[int] = None, step: int = 0,
                index0: int = 0) -> None:
    """SGD with momentum on the clipped gradient, in place on fp32 theta and on m (fp32, or uint16 = bfloat16)."""
    p, bf = _grad_ptr(g)
    if _is_bf16_state(theta, (m,), g.size):
        lib().adagc_ref_sgdm_bf16state(theta.ctypes.data, p, bf, m.ctypes.data, g.size, float(h), lr, momentum, wd,
                                       _tie_ptr(near_tie, g.size), float(tie_tol), int(fp32_decision),
                                       int(stochastic_seed is not None), int(stochastic_seed or 0), int(step), int(index0))
    else:
        lib().adagc_ref_sgdm(theta.ctypes.data, p, bf, m.ctypes.data, g.size, float(h), lr, momentum, wd)


def scale(g: np.ndarray, h: float, out: Optional[np.ndarray] = None) -> np.ndarray:
    """hat(g) = h * g rounded to the gradient's dtype."""
    p, bf = _grad_ptr(g)
    out = np.empty_like(g) if out is None else out
    lib().adagc_ref_scale(out.ctypes.data, p, bf, g.size, float(h))
    return out


def philox4x32_10(counter, key) -> np.ndarray:
    c, k, out = np.asarray(counter, np.uint32).copy(), np.asarray(key, np.uint32).copy(), np.zeros(4, np.uint32)
    lib().adagc_ref_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def float_to_bf16_stochastic_bits(x: float, r: int) -> int:
    return int(lib().adagc_ref_float_to_bf16_stochastic(float(np.float32(x)), int(r)))


def double_to_bf16_bits(x: float) -> int:
    return int(lib().adagc_ref_double_to_bf16(float(x)))


class ArenaOracle:
    """Algorithm 1 over tensors stored at fixed offsets of shared fp32 arenas (theta, m, v)."""

    def __init__(self, offsets: Sequence[int], numels: Sequence[int], theta0: np.ndarray, *,
                 lr: float, beta1: float, beta2: float, eps: float, wd: float, lambda_rel: float,
                 beta: float, lambda_abs: float, warmup: int, keep_initial: bool = False,
                 global_adaptive: bool = False, gamma0: Optional[np.ndarray] = None, ema_cap: float = 0.0,
                 bf16_state: bool = False, tie_tol: float = 0.0, fp32_decision: bool = False,
                 stochastic_seed: Optional[int] = None):
        """bf16_state: m and v are stored as bfloat16 (uint16 bit patterns), rounded to nearest even on store;
        `self.ties` then counts, per element, the steps whose float64 rounding was decided with a margin below
        tie_tol; fp32_decision: the rounded value is evaluated in single precision (see adagc_ref.c)."""
        self.fp32_decision = bool(fp32_decision)
        self.stochastic_seed = stochastic_seed
        self.keep_initial, self.global_adaptive, self.ema_cap = keep_initial, global_adaptive, float(ema_cap)
        self.bf16_state, self.tie_tol = bool(bf16_state), float(tie_tol)
        self.off = np.ascontiguousarray(offsets, dtype=np.int64)
        self.numel = np.ascontiguousarray(numels, dtype=np.int64)
        self.T = len(self.off)
        self.theta = np.array(theta0, dtype=np.float32)
        self.m = np.zeros(self.theta.shape, np.uint16 if bf16_state else np.float32)
        self.v = np.zeros_like(self.m)
        self.ties = np.zeros(self.theta.shape, np.uint8) if bf16_state else None
        self.gamma = np.zeros(self.T, dtype=np.float32) if gamma0 is None else np.array(gamma0, dtype=np.float32)
        self.hp = dict(lr=lr, beta1=beta1, beta2=beta2, eps=eps, wd=wd, lambda_rel=lambda_rel,
                       beta=beta, lambda_abs=lambda_abs, warmup=warmup)
        self.t = 0
        self.clip_count = np.zeros(self.T, dtype=np.uint64)
        self._s = np.empty(self.T, np.float64)

    def step(self, grads: np.ndarray, lr: Optional[float] = None):
        if self.keep_initial or self.global_adaptive or self.ema_cap > 0 or self.bf16_state:
            return self._step_variant(grads, lr)
        self.t += 1
        p, bf = _grad_ptr(grads)
        hp = self.hp
        norm, h, clipped, margin = (np.empty(self.T, np.float64) for _ in range(4))
        flag = np.empty(self.T, np.uint8)
        G = np.empty(1, np.float64)
        lib().adagc_ref_step(self.T, self.off, self.numel, self.theta.ctypes.data, p, bf,
                             self.m.ctypes.data, self.v.ctypes.data, self.gamma, self.t,
                             hp["lr"] if lr is None else lr, hp["beta1"], hp["beta2"], hp["eps"], hp["wd"],
                             hp["lambda_rel"], hp["beta"], hp["lambda_abs"], hp["warmup"],
                             self._s, norm, h, flag, clipped, margin, G)
        self.clip_count += flag.astype(np.uint64)
        return dict(norm=norm, h=h, flag=flag.astype(bool), clipped=clipped, margin=margin,
                    global_norm=float(G[0]), gamma=self.gamma.copy())

    def _step_variant(self, grads: np.ndarray, lr: Optional[float]):
        """One step with an ablation variant: the same three stages, composed from the single functions."""
        r = self.clip(grads)
        hp = self.hp
        for i in range(self.T):
            o, n = int(self.off[i]), int(self.numel[i])
            args = (self.theta[o:o + n], grads[o:o + n], self.m[o:o + n], self.v[o:o + n], float(r["h"][i]),
                    self.t, hp["lr"] if lr is None else lr, hp["beta1"], hp["beta2"], hp["eps"], hp["wd"])
            if self.bf16_state:
                adamw_update_bf16state(*args, near_tie=self.ties[o:o + n], tie_tol=self.tie_tol,
                                       fp32_decision=self.fp32_decision, stochastic_seed=self.stochastic_seed, index0=o)
            else:
                adamw_update(*args)
        return r

    def clip(self, grads: np.ndarray):
        """Clip-only step: advances gamma and the counters, returns the decisions (no AdamW)."""
        self.t += 1
        s = sumsq_tensors(grads, self.off, self.numel)
        r = clip_decisions(s, self.gamma, self.t, self.hp["lambda_rel"], self.hp["beta"],
                           self.hp["lambda_abs"], self.hp["warmup"], self.keep_initial, self.global_adaptive,
                           self.ema_cap)
        self.clip_count += r["flag"].astype(np.uint64)
        r["gamma"] = self.gamma.copy()
        return r
