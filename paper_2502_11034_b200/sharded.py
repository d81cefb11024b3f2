"""The fused step for a model whose tensors are sharded over several GPUs (flat equal shards).

Section 4.3 ("Communication") of the paper: once a tensor is split over devices, its norm needs one
all-reduce of the partial sums of squares inside the group that holds it -- and nothing else of the step
crosses devices.  Here every rank owns one contiguous range of the flat arenas; a step is

    adagc_shard_sumsq  ->  all-reduce of n_tensors float64 values (NCCL)  ->  adagc_step_presummed

with gamma replicated on every rank.  All arithmetic runs in the library's kernels; this module only plans
the shards (adagc_shard_plan), owns the n_tensors-long exchange buffer and calls torch.distributed.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch
import torch.distributed as dist

from . import binding


class ShardedAdaGC:
    """One rank's context over its slices of the tensors.

    The rank's arenas (params, grads, m, v) hold elements [elem_begin, elem_end) of the full arenas;
    `ema` has n_tensors entries on every rank."""

    def __init__(self, numels: Sequence[int], offsets: Sequence[int], grad_dtype: torch.dtype, lambda_abs: float,
                 rank: int, world: int, device="cuda", flags: int = 0, group=None):
        gd = {torch.float32: binding.ADAGC_F32, torch.bfloat16: binding.ADAGC_BF16}[grad_dtype]
        self.rank, self.world, self.group = int(rank), int(world), group
        self.local_numels, self.local_offsets, self.elem_begin, self.elem_end = binding.shard_plan(
            numels, offsets, gd, rank, world)
        self.n_tensors = len(numels)
        self.opt = binding.AdaGC(self.local_numels, self.local_offsets, grad_dtype, lambda_abs, device=device,
                                 flags=flags | binding.ALLOW_EMPTY)
        self.sumsq = torch.zeros(self.n_tensors, dtype=torch.float64, device=device)

    @property
    def local_elems(self) -> int:
        return self.elem_end - self.elem_begin

    def local_sumsq(self, grads_local: torch.Tensor, stream=None) -> torch.Tensor:
        """Phase 1 on this rank's gradient slice; returns the exchange buffer (not yet reduced)."""
        self.opt.shard_sumsq(grads_local, self.sumsq, stream)
        return self.sumsq

    def reduce(self) -> None:
        """Sum the exchange buffer over the ranks (the one exchange step of the path)."""
        if self.world > 1:
            dist.all_reduce(self.sumsq, op=dist.ReduceOp.SUM, group=self.group)

    def step(self, params, grads, m, v, ema, step, lr, beta1, beta2, eps, wd, lambda_rel, beta, warmup,
             stream=None):
        self.local_sumsq(grads, stream)
        self.reduce()
        self.opt.step_presummed(params, grads, m, v, ema, self.sumsq, step, lr, beta1, beta2, eps, wd,
                                lambda_rel, beta, warmup, stream)

    def clip(self, grads_in, grads_out, ema, step, lambda_rel, beta, warmup, stream=None):
        self.local_sumsq(grads_in, stream)
        self.reduce()
        self.opt.clip_presummed(grads_in, grads_out, ema, self.sumsq, step, lambda_rel, beta, warmup, stream)

    def close(self):
        self.opt.close()
