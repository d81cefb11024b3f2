"""The C-ABI library: it loads, exports every symbol the header declares, and its host-side
validation returns the documented error codes.  No kernel is launched here."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2502_11034_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(adagc_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    names = _declared_functions()
    assert {"adagc_create", "adagc_destroy", "adagc_step", "adagc_clip", "adagc_get_stats",
            "adagc_workspace_bytes", "adagc_step_host", "adagc_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"


def test_descriptor_validation_codes():
    lib = binding.lib()

    def chunks(numels, offsets, dt=binding.ADAGC_F32, lambda_abs=1.0, shapes=None, **kw):
        d, keep = binding.make_desc(numels, offsets, dt, lambda_abs, shapes, **kw)
        return int(lib.adagc_num_chunks(C.byref(d))), int(lib.adagc_workspace_bytes(C.byref(d)))

    assert chunks([16384, 16385, 1], [0, 16384, 32776]) [0] == 1 + 2 + 1
    assert chunks([100], [0], shapes=[(10, 10)])[0] == 1
    n, ws = chunks([100, 50], [0, 104], binding.ADAGC_BF16)
    assert n == 2 and ws > 0 and ws % 256 == 0
    assert chunks([], [])[0] == -1                                       # no tensors
    assert chunks([0], [0]) == (-1, 0)                                   # empty tensor
    assert chunks([-5], [0])[0] == -1
    assert chunks([100], [0], lambda_abs=0.0)[0] == -1
    assert chunks([100], [0], shapes=[(10, 11)])[0] == -1                # shape does not match numel
    assert chunks([100, 50], [0, 102])[0] == -2                          # fp32: offsets in multiples of 4
    assert chunks([100, 50], [0, 100], binding.ADAGC_BF16)[0] == -2      # bf16: multiples of 8
    assert chunks([(1 << 34) + 8], [0])[0] == -1                         # beyond the largest supported arena
    assert chunks([1 << 20], [(1 << 34) - 8])[0] == -1
    assert chunks([1 << 34], [0])[0] == (1 << 34) // 16384               # the maximum itself is accepted
    assert chunks([100, 50], [0, 96])[0] == -3                           # overlap
    assert chunks([50, 100], [96, 0])[0] == -3                           # overlap, unsorted
    assert chunks([100], [0], dt=2)[0] == -5
    assert chunks([100], [0], param_dtype=binding.ADAGC_BF16)[0] == -5
    assert chunks([100], [0], state_dtype=binding.ADAGC_BF16)[0] == 1                       # moments stored as bfloat16
    assert chunks([100], [0], state_dtype=2)[0] == -5
    assert chunks([100, 50], [0, 100], state_dtype=binding.ADAGC_BF16)[0] == -2            # then offsets in multiples of 8
    assert chunks([100], [0], flags=binding.SEPARATE_FINALIZE)[0] == 1
    assert chunks([100], [0], flags=binding.UPDATE_PATH_BULK)[0] == 1
    d, keep = binding.make_desc([8], [0], binding.ADAGC_F32)
    d.n_tensors = (1 << 24) + 1                                          # more tensors than the descriptor may list
    assert int(lib.adagc_num_chunks(C.byref(d))) == -1
    assert chunks([100], [0], flags=3)[0] == -1 and chunks([100], [0], flags=128)[0] == -1   # unknown flags
    assert chunks([100], [0], flags=binding.EMA_KEEP_INITIAL | binding.CLIP_GLOBAL_ADAPTIVE | 2)[0] == 1
    assert lib.adagc_workspace_bytes(None) == 0
    for code in range(-9, 1):
        assert binding.strerror(code) not in ("", "unknown status")
    assert binding.strerror(-99) == "unknown status"


def test_create_rejects_bad_workspace_and_null_out():
    lib = binding.lib()
    d, keep = binding.make_desc([100], [0], binding.ADAGC_F32)
    h = C.c_void_p()
    assert lib.adagc_create(C.byref(d), None, 1 << 20, None, C.byref(h)) == -4
    assert lib.adagc_create(C.byref(d), 256, 16, None, C.byref(h)) == -4          # too small
    assert lib.adagc_create(C.byref(d), 257, 1 << 20, None, C.byref(h)) == -4     # misaligned
    assert lib.adagc_create(C.byref(d), 256, 1 << 20, None, None) == -1
    assert lib.adagc_destroy(None) == -1
    assert lib.adagc_step(None, None, None, None, None, None, 1, 1e-3, .9, .95, 1e-8, .1, 1.04, .99, 0, None) == -1


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a GPU")
def test_no_cpu_fallback_without_a_device():
    """Without a CUDA device the product path must fail loudly, not compute on the CPU."""
    lib = binding.lib()
    d, keep = binding.make_desc([100], [0], binding.ADAGC_F32)
    h = C.c_void_p()
    assert lib.adagc_create(C.byref(d), 256, 1 << 24, None, C.byref(h)) == -6 and not h.value
    with pytest.raises(Exception):
        binding.AdaGC([100], [0], torch.float32)


def test_binding_and_oracle_do_not_import_each_other():
    pkg = os.path.join(ROOT, "paper_2502_11034_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, fn)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle|#include.*oracle|adagc_ref", text, flags=re.M), \
                    f"{fn} uses the oracle"
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2502_11034_b200" not in text and "adagc.h" not in text


def test_header_is_plain_c(tmp_path):
    """include/adagc.h must compile as C99 on its own (the boundary is a C ABI), and a C program that calls the
    host-only entry points links against the library and gets the documented answers."""
    import subprocess
    src = tmp_path / "use_adagc.c"
    src.write_text(r'''
#include "adagc.h"
#include <stdio.h>
int main(void) {
  adagc_tensor t[2] = {{0}};
  adagc_desc d = {0};
  adagc_tensor local[2];
  int64_t b = -1, e = -1;
  t[0].numel = 20000; t[0].offset = 0;
  t[1].numel = 100;   t[1].offset = 20000;
  d.n_tensors = 2; d.param_dtype = ADAGC_F32; d.grad_dtype = ADAGC_BF16; d.state_dtype = ADAGC_F32;
  d.tensors = t; d.lambda_abs = 1.0;
  if (adagc_num_chunks(&d) != 3) return 1;
  if (adagc_workspace_bytes(&d) == 0) return 2;
  if (adagc_shard_plan(&d, 1, 2, local, &b, &e) != ADAGC_OK) return 3;
  if (b != 10056 || e != 20100 || local[0].numel != 20000 - 10056 || local[1].numel != 100) return 4;
  d.lambda_abs = -1.0;
  if (adagc_num_chunks(&d) != ADAGC_E_INVALID_ARG) return 5;
  printf("%s\n", adagc_strerror(ADAGC_E_OVERLAP));
  return 0;
}
''')
    inc = os.path.join(ROOT, "include")
    libdir = os.path.join(ROOT, "paper_2502_11034_b200")
    binding.lib()                                           # the library exists (built by the build step)
    exe = tmp_path / "use_adagc"
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", inc, str(src), "-o", str(exe),
                    "-L", libdir, "-ladagc", f"-Wl,-rpath,{libdir}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, f"C program failed at check {out.returncode}"
    assert out.stdout.strip() == "tensors overlap"
