"""Seeded synthetic workloads: tensor layouts and per-step gradient streams.

This module serves both the CUDA path's tests/benchmarks and the CPU oracle's
tests.  It holds no arithmetic of the method itself (no norms, no clipping, no
optimizer update): only shapes, arena offsets, hyper-parameter presets and
random inputs.  Layouts follow the model shapes of the paper's hyper-parameter
table (Appendix "Hyper-Parameters": Llama-2 7B has 32 layers, hidden 4096,
FFN 11008) and the tensor census of Section 4.3 "Memory" (four attention
matrices, three FFN matrices and two norm vectors per dense layer, plus
embedding, final norm and LM head: 9*L + 3 tensors).

The paper trains on text corpora; here every gradient is a seeded random draw
with the shapes, dtypes and heavy-tail / spike structure of those runs.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

BASE_SEED = 20250211
ALIGN_ELEMS = 8  # every tensor starts on a 16-byte boundary in a bf16 arena (32 B in fp32)

# AdaGC / AdamW defaults of the paper's hyper-parameter table.
PAPER_DEFAULTS = dict(
    lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1,
    lambda_rel=1.04, beta=0.99, lambda_abs=1.0,
)


@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    numel: int
    offset: int  # element offset into every arena (params, grads, m, v)


@dataclass
class Workload:
    name: str
    config_id: int
    tensors: List[TensorSpec]
    grad_dtype: str  # "f32" | "bf16"
    hyper: Dict[str, float]
    warmup: int
    n_steps: int
    arena_elems: int
    grad_kind: str = "normal"  # "normal" | "student_t"
    grad_df: int = 0
    grad_scale: float = 1e-3
    per_tensor_std: Optional[np.ndarray] = None
    notes: str = ""
    extra: Dict[str, object] = field(default_factory=dict)

    @property
    def n_tensors(self) -> int:
        return len(self.tensors)

    @property
    def n_params(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def torch_grad_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.grad_dtype == "bf16" else torch.float32


def _layout(named_shapes: Sequence[Tuple[str, Tuple[int, ...]]]) -> Tuple[List[TensorSpec], int]:
    specs, off = [], 0
    for name, shape in named_shapes:
        n = int(np.prod(shape))
        specs.append(TensorSpec(name, tuple(int(s) for s in shape), n, off))
        off += (n + ALIGN_ELEMS - 1) // ALIGN_ELEMS * ALIGN_ELEMS
    return specs, off


# --------------------------------------------------------------------------- layouts
def tiny_mlp() -> Workload:
    shapes = [("fc1.w", (256, 512)), ("fc1.b", (512,)), ("fc2.w", (512, 512)), ("fc2.b", (512,)),
              ("fc3.w", (512, 256)), ("fc3.b", (256,)), ("out.w", (256, 10)), ("out.b", (10,))]
    specs, total = _layout(shapes)
    hyper = dict(PAPER_DEFAULTS, lr=1e-3, lambda_rel=1.05, beta=0.98)
    return Workload("tiny", 1, specs, "f32", hyper, warmup=3, n_steps=12, arena_elems=total,
                    grad_kind="normal", grad_scale=1e-3,
                    extra={"spike_step": 6, "spike_tensor": 3, "spike_factor": 100.0},
                    notes="2-layer-MLP-shaped, 8 fp32 tensors")


def gpt2_small(n_layer: int = 12, d: int = 768, vocab: int = 50257, n_pos: int = 1024) -> Workload:
    shapes: List[Tuple[str, Tuple[int, ...]]] = [("wte", (vocab, d)), ("wpe", (n_pos, d))]
    for l in range(n_layer):
        p = f"h{l}."
        shapes += [(p + "ln1.w", (d,)), (p + "ln1.b", (d,)),
                   (p + "attn.qkv.w", (d, 3 * d)), (p + "attn.qkv.b", (3 * d,)),
                   (p + "attn.proj.w", (d, d)), (p + "attn.proj.b", (d,)),
                   (p + "ln2.w", (d,)), (p + "ln2.b", (d,)),
                   (p + "mlp.fc.w", (d, 4 * d)), (p + "mlp.fc.b", (4 * d,)),
                   (p + "mlp.proj.w", (4 * d, d)), (p + "mlp.proj.b", (d,))]
    shapes += [("ln_f.w", (d,)), ("ln_f.b", (d,))]
    specs, total = _layout(shapes)
    rng = np.random.RandomState(BASE_SEED + 2000)
    std = np.exp(rng.uniform(math.log(1e-5), math.log(1e-2), size=len(specs)))
    return Workload("gpt2_small", 2, specs, "bf16", dict(PAPER_DEFAULTS), warmup=10, n_steps=50,
                    arena_elems=total, grad_kind="normal", grad_scale=1.0, per_tensor_std=std,
                    extra={"spike_frac": 0.01, "spike_factor": 50.0},
                    notes="GPT-2-small-shaped, tied embeddings, per-tensor log-uniform grad scale")


def llama_dense(name: str, config_id: int, n_layer: int, d: int, ffn: int, vocab: int,
                kv_dim: Optional[int] = None, tied: bool = False) -> List[Tuple[str, Tuple[int, ...]]]:
    kv = d if kv_dim is None else kv_dim
    shapes: List[Tuple[str, Tuple[int, ...]]] = [("embed", (vocab, d))]
    for l in range(n_layer):
        p = f"l{l}."
        shapes += [(p + "attn_norm", (d,)),
                   (p + "q_proj", (d, d)), (p + "k_proj", (kv, d)), (p + "v_proj", (kv, d)),
                   (p + "o_proj", (d, d)),
                   (p + "ffn_norm", (d,)),
                   (p + "gate_proj", (ffn, d)), (p + "up_proj", (ffn, d)), (p + "down_proj", (d, ffn))]
    shapes.append(("final_norm", (d,)))
    if not tied:
        shapes.append(("lm_head", (vocab, d)))
    return shapes


def llama2_7b(n_layer: int = 32, d: int = 4096, ffn: int = 11008, vocab: int = 32000) -> Workload:
    specs, total = _layout(llama_dense("llama2_7b", 3, n_layer, d, ffn, vocab))
    spiked = [i for i, t in enumerate(specs)
              if any(t.name == f"l{l}.{w}" for l in range(min(4, n_layer)) for w in ("q_proj", "k_proj"))]
    return Workload("llama2_7b", 3, specs, "bf16", dict(PAPER_DEFAULTS), warmup=5, n_steps=20,
                    arena_elems=total, grad_kind="normal", grad_scale=1e-4,
                    extra={"spike_step": 12, "spike_tensors": spiked, "spike_factor": 1000.0},
                    notes="Llama-2-7B-shaped: 9 tensors per layer + embed, final norm, lm_head")


def many_small(n_tensors: int = 20000, lo: int = 64, hi: int = 65536) -> Workload:
    rng = np.random.RandomState(BASE_SEED + 4000)
    sizes = np.rint(np.exp(rng.uniform(math.log(lo), math.log(hi), size=n_tensors))).astype(np.int64)
    specs, total = _layout([(f"t{i}", (int(n),)) for i, n in enumerate(sizes)])
    return Workload("many_small", 4, specs, "f32", dict(PAPER_DEFAULTS), warmup=5, n_steps=30,
                    arena_elems=total, grad_kind="student_t", grad_df=2, grad_scale=1e-3,
                    notes="log-uniform tensor sizes, Student-t(2) gradients")


def llama32_1b(n_layer: int = 16, d: int = 2048, ffn: int = 8192, vocab: int = 128256,
               kv_dim: int = 512) -> Workload:
    specs, total = _layout(llama_dense("llama32_1b", 5, n_layer, d, ffn, vocab, kv_dim=kv_dim, tied=True))
    return Workload("llama32_1b", 5, specs, "bf16", dict(PAPER_DEFAULTS), warmup=10, n_steps=100,
                    arena_elems=total, grad_kind="student_t", grad_df=3, grad_scale=1e-4,
                    extra={"spike_frac": 0.05, "spike_lo": 10.0, "spike_hi": 1000.0},
                    notes="Llama-3.2-1B-shaped, tied embedding, GQA k/v, Student-t(3) gradients")


def moe_8x1b(n_layer: int = 24, d: int = 2048, ffn: int = 5632, vocab: int = 32000, kv_dim: int = 256,
             n_experts: int = 8) -> Workload:
    """Mixture-of-experts layout shaped like the paper's Mixtral 8x1B run (hyper-parameter table: 24 layers,
    hidden 2048, FFN 5632, 32 heads, 4 key-value heads, 8 routed experts).  Per layer: four attention
    matrices, a router, three matrices per expert and two norm vectors, i.e. (7 + 3E) L + 3 tensors -- the
    census of Section 4.3 "Memory" with no shared expert and the router counted."""
    shapes: List[Tuple[str, Tuple[int, ...]]] = [("embed", (vocab, d))]
    for l in range(n_layer):
        p = f"l{l}."
        shapes += [(p + "attn_norm", (d,)), (p + "q_proj", (d, d)), (p + "k_proj", (kv_dim, d)),
                   (p + "v_proj", (kv_dim, d)), (p + "o_proj", (d, d)), (p + "ffn_norm", (d,)),
                   (p + "router", (n_experts, d))]
        for e in range(n_experts):
            shapes += [(p + f"e{e}.gate_proj", (ffn, d)), (p + f"e{e}.up_proj", (ffn, d)),
                       (p + f"e{e}.down_proj", (d, ffn))]
    shapes += [("final_norm", (d,)), ("lm_head", (vocab, d))]
    specs, total = _layout(shapes)
    hyper = dict(PAPER_DEFAULTS, beta2=0.999)          # the table's Adam beta2 for this model
    return Workload("moe_8x1b", 6, specs, "bf16", hyper, warmup=5, n_steps=20, arena_elems=total,
                    grad_kind="student_t", grad_df=3, grad_scale=1e-4,
                    extra={"spike_frac": 0.02, "spike_lo": 10.0, "spike_hi": 1000.0},
                    notes="Mixtral-8x1B-shaped MoE: (7+3E)L+3 tensors, experts get heavy-tailed gradients")


def moe_ernie(n_layer: int = 25, d: int = 2560, ffn: int = 1024, vocab: int = 32000, kv_dim: int = 512,
              n_experts: int = 48, n_shared: int = 1) -> Workload:
    """Fine-grained mixture-of-experts layout shaped like the paper's ERNIE 10B-A1.4B run (hyper-parameter
    table: 25 layers, hidden 2560, expert FFN 1024, 20 heads, 4 key-value heads of 128, one shared and 48
    routed experts).  Tensor census exactly as Section 4.3 "Memory" counts it: per layer four attention
    matrices, three matrices for each of the 1 + E experts and two norm vectors, plus embedding, final norm
    and LM head: (9 + 3E) L + 3 = 3828 tensors.  The vocabulary size is not given in the paper; 32000 is
    assumed (it only sets the size of two tensors)."""
    shapes: List[Tuple[str, Tuple[int, ...]]] = [("embed", (vocab, d))]
    for l in range(n_layer):
        p = f"l{l}."
        shapes += [(p + "attn_norm", (d,)), (p + "q_proj", (d, d)), (p + "k_proj", (kv_dim, d)),
                   (p + "v_proj", (kv_dim, d)), (p + "o_proj", (d, d)), (p + "ffn_norm", (d,))]
        for e in range(n_shared + n_experts):
            tag = f"s{e}" if e < n_shared else f"e{e - n_shared}"
            shapes += [(p + tag + ".gate_proj", (ffn, d)), (p + tag + ".up_proj", (ffn, d)),
                       (p + tag + ".down_proj", (d, ffn))]
    shapes += [("final_norm", (d,)), ("lm_head", (vocab, d))]
    specs, total = _layout(shapes)
    return Workload("moe_ernie", 7, specs, "bf16", dict(PAPER_DEFAULTS), warmup=5, n_steps=20, arena_elems=total,
                    grad_kind="student_t", grad_df=3, grad_scale=1e-4,
                    extra={"spike_frac": 0.01, "spike_lo": 10.0, "spike_hi": 1000.0},
                    notes="ERNIE-10B-A1.4B-shaped MoE: (9+3E)L+3 tensors, 2.6 M-element expert matrices")


_BUILDERS = {"tiny": tiny_mlp, "moe_8x1b": moe_8x1b, "moe_ernie": moe_ernie, "gpt2_small": gpt2_small, "llama2_7b": llama2_7b,
             "many_small": many_small, "llama32_1b": llama32_1b}


def build(name: str, **overrides) -> Workload:
    """Build a named layout; keyword overrides shrink it (e.g. n_layer=2, d=256) for small tests."""
    return _BUILDERS[name](**overrides)


# --------------------------------------------------------------------------- random inputs
def _generator(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def step_seed(wl: Workload, step: int) -> int:
    return BASE_SEED + 1000 * wl.config_id + int(step)


def init_params(wl: Workload, device="cpu", std: float = 0.02) -> torch.Tensor:
    """theta_0 arena (fp32), N(0, std); padding gaps are zero."""
    gen = _generator(device, BASE_SEED + 1000 * wl.config_id)
    theta = torch.empty(wl.arena_elems, dtype=torch.float32, device=device)
    theta.normal_(0.0, std, generator=gen)
    _zero_padding(wl, theta)
    return theta


def _zero_padding(wl: Workload, arena: torch.Tensor) -> None:
    if wl.arena_elems == wl.n_params:
        return
    starts = np.array([t.offset + t.numel for t in wl.tensors], dtype=np.int64)
    ends = np.array([t.offset for t in wl.tensors[1:]] + [wl.arena_elems], dtype=np.int64)
    gaps = np.nonzero(ends > starts)[0]
    if len(gaps) == 0:
        return
    idx = np.concatenate([np.arange(starts[k], ends[k]) for k in gaps])
    arena[torch.from_numpy(idx).to(arena.device)] = 0


def spikes_for_step(wl: Workload, step: int) -> List[Tuple[int, float]]:
    """(tensor index, multiplier) pairs injected at this 1-based step."""
    ex = wl.extra
    if "spike_step" in ex:
        if step != ex["spike_step"]:
            return []
        idx = ex.get("spike_tensors", [ex.get("spike_tensor")])
        return [(int(i), float(ex["spike_factor"])) for i in idx]
    if "spike_frac" in ex:
        rng = np.random.RandomState(step_seed(wl, step) % (2 ** 31))
        k = max(1, int(round(ex["spike_frac"] * wl.n_tensors)))
        idx = rng.permutation(wl.n_tensors)[:k]
        if "spike_factor" in ex:
            fac = np.full(k, float(ex["spike_factor"]))
        else:
            fac = np.exp(rng.uniform(math.log(ex["spike_lo"]), math.log(ex["spike_hi"]), size=k))
        return [(int(i), float(f)) for i, f in zip(idx, fac)]
    return []


def _student_t(n: int, df: int, gen: torch.Generator, device) -> torch.Tensor:
    z = torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen)
    chi2 = torch.zeros(n, dtype=torch.float32, device=device)
    tmp = torch.empty(n, dtype=torch.float32, device=device)
    for _ in range(df):
        tmp.normal_(0.0, 1.0, generator=gen)
        chi2.addcmul_(tmp, tmp)
    del tmp
    chi2.div_(df).sqrt_().clamp_(min=1e-20)
    z.div_(chi2)
    return z


def grads_for_step(wl: Workload, step: int, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Gradient arena for a 1-based step, in the workload's gradient dtype.

    The same (workload, step, device type) always yields the same bits; the CUDA
    path and the oracle are fed the same tensor (copied, never regenerated on
    another device type).
    """
    gen = _generator(device, step_seed(wl, step))
    dt = wl.torch_grad_dtype
    g = out if out is not None else torch.empty(wl.arena_elems, dtype=dt, device=device)
    assert g.dtype == dt and g.numel() == wl.arena_elems
    if wl.grad_kind == "normal" and wl.per_tensor_std is None:
        g.normal_(0.0, wl.grad_scale, generator=gen)
    elif wl.grad_kind == "normal":
        for t, s in zip(wl.tensors, wl.per_tensor_std):
            g[t.offset:t.offset + t.numel].normal_(0.0, float(s) * wl.grad_scale, generator=gen)
    elif wl.grad_kind == "student_t":
        block = 1 << 26
        for lo in range(0, wl.arena_elems, block):
            n = min(block, wl.arena_elems - lo)
            g[lo:lo + n] = (_student_t(n, wl.grad_df, gen, device) * wl.grad_scale).to(dt)
    else:
        raise ValueError(wl.grad_kind)
    for i, fac in spikes_for_step(wl, step):
        t = wl.tensors[i]
        view = g[t.offset:t.offset + t.numel]
        view.copy_((view.float() * fac).to(dt))
    _zero_padding(wl, g)
    return g
