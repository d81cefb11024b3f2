"""The bounds-checked build of the library (-DADAGC_BOUNDS_CHECK): every kernel verifies the chunk-table entries it is
about to walk and would set ADAGC_E_BOUNDS instead of touching memory.  Here the ragged and many-small-tensor cases (and
one run of each other entry point) go through that build in a child process and must give the oracle's results with a
clean status word, i.e. the checks never fire on tables that adagc_create wrote."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r}); sys.path.insert(0, {root!r} + "/tests")
import torch
from paper_2502_11034_b200 import binding, workloads
import parity_harness as H
from test_gpu_parity import _ragged_workload
assert binding.lib().adagc_debug_bounds_checked_build() == 1, "the checked library was not loaded"
sizes = [1, 2, 3, 5, 7, 8, 9, 10, 15, 16, 17, 31, 33, 255, 257, 2047, 2049, 16383, 16384, 16385, 32767, 32768, 32769,
         3 * 16384 + 5, 100003, 40 * 16384, 9 * 16384 + 4095]
for dtype in ("f32", "bf16"):
    wl = _ragged_workload(sizes, dtype)
    for flags in (binding.UPDATE_PATH_REGISTERS, binding.UPDATE_PATH_BULK, binding.SEPARATE_FINALIZE, binding.FUSED_SMALL):
        H.run_full(wl, 6, flags=flags)                      # asserts status == 0 at the end
    H.run_full_clip(wl, 4, in_place=True)
    H.run_full_clip(wl, 4, in_place=False)
    H.run_full_lion(wl, 4)
    H.run_bf16_state(wl, 4)
    H.run_full_sharded(wl, 4, 3)
wl = workloads.build("many_small", n_tensors=3000, lo=16, hi=40000)
H.run_full(wl, 6, hyper_over=dict(lambda_abs=1e4))
H.run_bf16_state(wl, 3, teacher_forced=True, hyper_over=dict(lambda_abs=1e4))   # partial chunks through the ring
H.run_bf16_state(wl, 3, hyper_over=dict(lambda_abs=1e4), stochastic_seed=5)
H.run_full(workloads.build("tiny"), 12)
print("checked build ok")
"""


def test_ragged_and_many_small_cases_on_the_checked_build():
    from paper_2502_11034_b200 import build
    lib = build.build(checked=True)
    env = dict(os.environ, ADAGC_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT)], env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0 and "checked build ok" in r.stdout, (r.stdout[-2000:], r.stderr[-4000:])
