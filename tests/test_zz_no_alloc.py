"""adagc_sumsq_noalloc: the entry point for callers that cannot allocate device memory (code that runs
while an allocator is locked or exhausted, plug-ins that only get their input and output buffers).
It must agree with the sums of squares that the regular, workspace-based path produces, on two calls
in a row (the calls share one fixed scratch array that keeps the previous call's contents).

This file is collected last on purpose: a run that stops at the first failure has then already run
every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2502_11034_b200 import binding

pytestmark = pytest.mark.gpu

RTOL = 1e-11          # the tolerance the parity tests use for float64 sums of squares


def _regular_sumsq(g: torch.Tensor) -> float:
    """The existing path: one-tensor descriptor, caller-allocated workspace, norm phase of adagc_clip."""
    opt = binding.AdaGC([g.numel()], [0], g.dtype, 1.0)
    ema = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = torch.empty_like(g)
    opt.clip(g, out, ema, 1, 1.04, 0.99, 0)
    s = float(opt.get_sumsq()[0])
    opt.close()
    return s


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_two_calls_in_a_row_match_the_workspace_path(dtype):
    gen = torch.Generator("cuda").manual_seed(123)
    big = (torch.randn(5 * 16384 + 13, device="cuda", generator=gen) * 1e-2).to(dtype)      # 6 chunks, ragged tail
    small = (torch.randn(16384 + 3, device="cuda", generator=gen) * 3.0).to(dtype)          # 2 chunks: stale partials
    want_big, want_small = _regular_sumsq(big), _regular_sumsq(small)                        # beyond them must not leak
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    side = torch.cuda.Stream()                                    # an explicit, non-default stream
    binding.sumsq_noalloc(small, out[1:2])                        # first call on this device: looks up the array's address
    torch.cuda.synchronize()
    # free device memory as the driver counts it (torch's own counters would not see a cudaMalloc inside the library)
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    side.wait_stream(torch.cuda.current_stream())
    binding.sumsq_noalloc(big, out[0:1], stream=side)
    binding.sumsq_noalloc(small, out[1:2], stream=side)
    side.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
    got = out.cpu().numpy()
    assert got[0] == pytest.approx(want_big, rel=RTOL)
    assert got[1] == pytest.approx(want_small, rel=RTOL)
    # and against plain float64 arithmetic on the host
    assert got[0] == pytest.approx(float((big.double().cpu() ** 2).sum()), rel=1e-12)
    assert got[1] == pytest.approx(float((small.double().cpu() ** 2).sum()), rel=1e-12)
    # a third call on the first buffer reproduces the first result bit for bit
    binding.sumsq_noalloc(big, out[1:2])
    assert float(out[1]) == got[0]


def test_limits_and_argument_errors():
    lib = binding.lib()
    g = torch.ones(64, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    too_many = (1 << 30) + 1
    assert lib.adagc_sumsq_noalloc(g.data_ptr(), binding.ADAGC_F32, too_many, out.data_ptr(), None) == -8
    assert "scratch" in binding.strerror(-8)
    assert lib.adagc_sumsq_noalloc(g.data_ptr(), binding.ADAGC_F32, 0, out.data_ptr(), None) == -1
    assert lib.adagc_sumsq_noalloc(None, binding.ADAGC_F32, 64, out.data_ptr(), None) == -1
    assert lib.adagc_sumsq_noalloc(g.data_ptr(), 7, 64, out.data_ptr(), None) == -5
    assert lib.adagc_sumsq_noalloc(g.data_ptr() + 4, binding.ADAGC_F32, 60, out.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert float(out[0]) == 0.0                                   # rejected calls enqueue nothing
    binding.sumsq_noalloc(g, out)
    assert float(out[0]) == 64.0
