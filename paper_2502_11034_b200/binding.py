"""ctypes binding of the C ABI in include/adagc.h (argument marshalling only).

PyTorch appears here only as the owner of device memory and streams: tensors are passed to
the library as raw device pointers, the current CUDA stream as a void*.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

ADAGC_F32, ADAGC_BF16 = 0, 1
ADAGC_W_NONFINITE = 1
ADAGC_E_TIMEOUT = 2
ADAGC_E_BOUNDS = 4
UPDATE_PATH_AUTO, UPDATE_PATH_REGISTERS, UPDATE_PATH_BULK = 0, 1, 2
EMA_KEEP_INITIAL, CLIP_GLOBAL_ADAPTIVE, ALLOW_EMPTY, FUSED_SMALL, SEPARATE_FINALIZE = 4, 8, 16, 32, 64

# ADAGC_LIBRARY selects another build of the same library (e.g. the bounds-checked one, libadagc_checked.so)
_LIB_PATH = os.environ.get("ADAGC_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libadagc.so")
_lib = None


class AdagcError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: adagc status {status} ({strerror(status)})")


class adagc_tensor(C.Structure):
    _fields_ = [("numel", C.c_int64), ("offset", C.c_int64), ("ndim", C.c_int32),
                ("reserved", C.c_int32), ("shape", C.c_int64 * 4)]


class adagc_desc(C.Structure):
    _fields_ = [("n_tensors", C.c_int32), ("param_dtype", C.c_int32), ("grad_dtype", C.c_int32),
                ("state_dtype", C.c_int32), ("tensors", C.POINTER(adagc_tensor)),
                ("lambda_abs", C.c_double), ("flags", C.c_int32), ("reserved", C.c_int32)]


def lib() -> C.CDLL:
    """Load libadagc.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2502_11034_b200.build` "
                          "(or __graft_entry__.build()); this package has no CPU fallback")
    L = C.CDLL(_LIB_PATH)
    vp, i64, dbl, f32p = C.c_void_p, C.c_int64, C.c_double, C.c_void_p
    L.adagc_workspace_bytes.restype = C.c_size_t
    L.adagc_workspace_bytes.argtypes = [C.POINTER(adagc_desc)]
    L.adagc_num_chunks.restype = i64
    L.adagc_num_chunks.argtypes = [C.POINTER(adagc_desc)]
    L.adagc_create.restype = C.c_int
    L.adagc_create.argtypes = [C.POINTER(adagc_desc), vp, C.c_size_t, vp, C.POINTER(vp)]
    L.adagc_destroy.restype = C.c_int
    L.adagc_destroy.argtypes = [vp]
    L.adagc_step.restype = C.c_int
    L.adagc_step.argtypes = [vp, vp, vp, vp, vp, f32p, i64, dbl, dbl, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_step_capturable.restype = C.c_int
    L.adagc_step_capturable.argtypes = [vp, vp, vp, vp, vp, f32p, vp, dbl, dbl, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_set_step_counter.restype = C.c_int
    L.adagc_set_step_counter.argtypes = [vp, C.c_uint64, vp]
    L.adagc_step_emit_bf16.restype = C.c_int
    L.adagc_step_emit_bf16.argtypes = [vp, vp, vp, vp, vp, vp, f32p, i64, dbl, dbl, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_step_lion.restype = C.c_int
    L.adagc_step_lion.argtypes = [vp, vp, vp, vp, f32p, i64, dbl, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_step_sgdm.restype = C.c_int
    L.adagc_step_sgdm.argtypes = [vp, vp, vp, vp, f32p, i64, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_clip.restype = C.c_int
    L.adagc_clip.argtypes = [vp, vp, vp, f32p, i64, dbl, dbl, i64, vp]
    L.adagc_step_host.restype = C.c_int
    L.adagc_step_host.argtypes = [vp, vp, vp, vp, vp, f32p, vp, i64, dbl, dbl, dbl, dbl, dbl, dbl, dbl, i64,
                                  vp, vp, vp, vp]
    L.adagc_shard_sumsq.restype = C.c_int
    L.adagc_shard_sumsq.argtypes = [vp, vp, vp, vp]
    L.adagc_step_presummed.restype = C.c_int
    L.adagc_step_presummed.argtypes = [vp, vp, vp, vp, vp, f32p, vp, i64, dbl, dbl, dbl, dbl, dbl, dbl, dbl, i64, vp]
    L.adagc_clip_presummed.restype = C.c_int
    L.adagc_clip_presummed.argtypes = [vp, vp, vp, f32p, vp, i64, dbl, dbl, i64, vp]
    L.adagc_shard_plan.restype = C.c_int
    L.adagc_shard_plan.argtypes = [C.POINTER(adagc_desc), C.c_int32, C.c_int32, C.POINTER(adagc_tensor),
                                   C.POINTER(i64), C.POINTER(i64)]
    L.adagc_get_stats.restype = C.c_int
    L.adagc_get_stats.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.adagc_get_sumsq.restype = C.c_int
    L.adagc_get_sumsq.argtypes = [vp, vp, vp]
    L.adagc_set_ema_cap.restype = C.c_int
    L.adagc_set_ema_cap.argtypes = [vp, dbl]
    L.adagc_set_state_rounding.restype = C.c_int
    L.adagc_set_state_rounding.argtypes = [vp, C.c_int32, C.c_uint64]
    L.adagc_update_path.restype = C.c_int
    L.adagc_update_path.argtypes = [vp]
    L.adagc_launch_grids.restype = C.c_int
    L.adagc_launch_grids.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    L.adagc_arena_elems.restype = i64
    L.adagc_arena_elems.argtypes = [vp]
    L.adagc_launch_count.restype = C.c_uint64
    L.adagc_launch_count.argtypes = [vp]
    L.adagc_set_phase_timing.restype = C.c_int
    L.adagc_set_phase_timing.argtypes = [vp, C.c_int]
    L.adagc_get_phase_times.restype = C.c_int
    L.adagc_get_phase_times.argtypes = [vp, C.POINTER(C.c_float)]
    L.adagc_sumsq_noalloc.restype = C.c_int
    L.adagc_sumsq_noalloc.argtypes = [vp, C.c_int32, i64, vp, vp]
    L.adagc_debug_wait_timeout.restype = C.c_int
    L.adagc_debug_wait_timeout.argtypes = [vp, dbl, vp]
    L.adagc_debug_chunk_tables.restype = C.c_int
    L.adagc_debug_chunk_tables.argtypes = [C.POINTER(adagc_desc), C.c_int32, C.c_int32, vp, vp, vp, vp, vp, vp]
    L.adagc_debug_chunk_entry_ok.restype = C.c_int
    L.adagc_debug_chunk_entry_ok.argtypes = [i64, C.c_int32, C.c_int32, C.c_int32, i64, C.c_int32, C.c_int32]
    L.adagc_debug_bounds_checked_build.restype = C.c_int
    L.adagc_debug_bounds_checked_build.argtypes = []
    L.adagc_debug_latch_status.restype = C.c_int
    L.adagc_debug_latch_status.argtypes = [vp, C.c_int32]
    L.adagc_strerror.restype = C.c_char_p
    L.adagc_strerror.argtypes = [C.c_int]
    _lib = L
    return L


def strerror(status: int) -> str:
    return lib().adagc_strerror(int(status)).decode()


def sumsq_noalloc(grads: torch.Tensor, out: torch.Tensor, numel: Optional[int] = None, stream=None) -> None:
    """adagc_sumsq_noalloc: sum of squares of a contiguous gradient buffer into `out` (one float64 on the
    device) without any workspace; for callers that cannot allocate device memory.  Enqueues only."""
    gd = {torch.float32: ADAGC_F32, torch.bfloat16: ADAGC_BF16}[grads.dtype]
    assert out.dtype == torch.float64 and out.is_cuda and grads.is_cuda and grads.is_contiguous()
    n = grads.numel() if numel is None else int(numel)
    with torch.cuda.device(grads.device):
        rc = lib().adagc_sumsq_noalloc(_ptr(grads), gd, n, _ptr(out), _stream_ptr(stream))
    if rc != 0:
        raise AdagcError(rc, "adagc_sumsq_noalloc")


def make_desc(numels: Sequence[int], offsets: Sequence[int], grad_dtype: int, lambda_abs: float = 1.0,
              shapes: Optional[Sequence[Sequence[int]]] = None, param_dtype: int = ADAGC_F32,
              state_dtype: int = ADAGC_F32, flags: int = 0):
    """Build an adagc_desc; returns (desc, keepalive) -- keep both alive while the desc is used."""
    n = len(numels)
    arr = (adagc_tensor * max(n, 1))()
    for i in range(n):
        arr[i].numel, arr[i].offset = int(numels[i]), int(offsets[i])
        shp = tuple(shapes[i]) if shapes is not None else ()
        if 0 < len(shp) <= 4:
            arr[i].ndim = len(shp)
            for k, s in enumerate(shp):
                arr[i].shape[k] = int(s)
    d = adagc_desc()
    d.n_tensors, d.param_dtype, d.grad_dtype, d.state_dtype = n, param_dtype, grad_dtype, state_dtype
    d.tensors = C.cast(arr, C.POINTER(adagc_tensor))
    d.lambda_abs = float(lambda_abs)
    d.flags = int(flags)
    return d, arr


def chunk_tables(numels: Sequence[int], offsets: Sequence[int], grad_dtype: int, which: int, grid: int,
                 state_dtype: int = ADAGC_F32, flags: int = 0):
    """adagc_debug_chunk_tables: dict(start, count, tensor, partial, block_begin[, block_mid]) of numpy arrays; host-only."""
    d, keep = make_desc(numels, offsets, grad_dtype, state_dtype=state_dtype, flags=flags)
    n = int(lib().adagc_num_chunks(C.byref(d)))
    if n < 0:
        raise AdagcError(n, "invalid descriptor")
    out = dict(start=np.zeros(n, np.int64), count=np.zeros(n, np.int32), tensor=np.zeros(n, np.int32),
               partial=np.zeros(n, np.int32), block_begin=np.zeros(grid + 1, np.int32), block_mid=np.zeros(grid, np.int32))
    rc = lib().adagc_debug_chunk_tables(C.byref(d), int(which), int(grid), *(out[k].ctypes.data for k in
                                        ("start", "count", "tensor", "partial", "block_begin", "block_mid")))
    if rc != 0:
        raise AdagcError(rc, "adagc_debug_chunk_tables")
    return out


def shard_plan(numels: Sequence[int], offsets: Sequence[int], grad_dtype: int, rank: int, world: int):
    """adagc_shard_plan: this rank's slice of every tensor under flat equal shards.
    Returns (local_numels, local_offsets, elem_begin, elem_end); host-only."""
    d, keep = make_desc(numels, offsets, grad_dtype)
    out = (adagc_tensor * max(len(numels), 1))()
    b, e = C.c_int64(), C.c_int64()
    rc = lib().adagc_shard_plan(C.byref(d), int(rank), int(world), out, C.byref(b), C.byref(e))
    if rc != 0:
        raise AdagcError(rc, "adagc_shard_plan")
    n = len(numels)
    return [int(out[i].numel) for i in range(n)], [int(out[i].offset) for i in range(n)], int(b.value), int(e.value)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


class AdaGC:
    """adagc_ctx plus its torch-owned workspace.  Method names mirror the C entry points."""

    def __init__(self, numels: Sequence[int], offsets: Sequence[int], grad_dtype: torch.dtype,
                 lambda_abs: float = 1.0, shapes=None, device="cuda", flags: int = 0,
                 state_dtype: torch.dtype = torch.float32):
        L = lib()
        gd = {torch.float32: ADAGC_F32, torch.bfloat16: ADAGC_BF16}[grad_dtype]
        self.grad_dtype = grad_dtype
        self.state_dtype = state_dtype           # dtype of the m and v arenas (adagc_desc.state_dtype)
        self.n_tensors = len(numels)
        self.device = torch.device(device)
        desc, keep = make_desc(numels, offsets, gd, lambda_abs, shapes, flags=flags,
                               state_dtype={torch.float32: ADAGC_F32, torch.bfloat16: ADAGC_BF16}[state_dtype])
        nbytes = L.adagc_workspace_bytes(C.byref(desc))
        if nbytes == 0:
            rc = L.adagc_num_chunks(C.byref(desc))
            raise AdagcError(int(rc), "invalid descriptor")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        assert self.workspace.data_ptr() % 256 == 0
        self.n_chunks = int(L.adagc_num_chunks(C.byref(desc)))
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = L.adagc_create(C.byref(desc), self.workspace.data_ptr(), nbytes, _stream_ptr(None), C.byref(h))
        if rc != 0:
            raise AdagcError(rc, "adagc_create")
        self._h = h
        self.arena_elems = int(L.adagc_arena_elems(h))
        self.update_path = int(L.adagc_update_path(h))

    def close(self):
        if getattr(self, "_h", None):
            lib().adagc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the entry points ------------------------------------------------------------------
    def step(self, params, grads, m, v, ema, step, lr, beta1, beta2, eps, wd, lambda_rel, beta, warmup,
             stream=None):
        assert grads.dtype == self.grad_dtype and params.dtype == ema.dtype == torch.float32 and m.dtype == v.dtype == self.state_dtype
        rc = lib().adagc_step(self._h, _ptr(params), _ptr(grads), _ptr(m), _ptr(v), _ptr(ema), int(step),
                              lr, beta1, beta2, eps, wd, lambda_rel, beta, int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step")

    def step_capturable(self, params, grads, m, v, ema, lr, beta1, beta2, eps, wd, lambda_rel, beta, warmup,
                        lr_dev: Optional[torch.Tensor] = None, stream=None):
        """adagc_step_capturable: the step number lives on the device; `lr_dev` (one fp32 on the device), if given,
        is read at every execution instead of `lr`."""
        assert grads.dtype == self.grad_dtype and params.dtype == ema.dtype == torch.float32 and m.dtype == v.dtype == self.state_dtype
        assert lr_dev is None or (lr_dev.dtype == torch.float32 and lr_dev.is_cuda)
        rc = lib().adagc_step_capturable(self._h, _ptr(params), _ptr(grads), _ptr(m), _ptr(v), _ptr(ema),
                                         _ptr(lr_dev), lr, beta1, beta2, eps, wd, lambda_rel, beta, int(warmup),
                                         _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_capturable")

    def set_step_counter(self, steps_done: int, stream=None):
        rc = lib().adagc_set_step_counter(self._h, int(steps_done), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_set_step_counter")

    def step_emit_bf16(self, params, params_bf16, grads, m, v, ema, step, lr, beta1, beta2, eps, wd, lambda_rel, beta,
                       warmup, stream=None):
        assert grads.dtype == self.grad_dtype and params_bf16.dtype == torch.bfloat16
        assert params.dtype == ema.dtype == torch.float32 and m.dtype == v.dtype == self.state_dtype
        rc = lib().adagc_step_emit_bf16(self._h, _ptr(params), _ptr(params_bf16), _ptr(grads), _ptr(m), _ptr(v),
                                        _ptr(ema), int(step), lr, beta1, beta2, eps, wd, lambda_rel, beta,
                                        int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_emit_bf16")

    def step_lion(self, params, grads, m, ema, step, lr, beta1, beta2, wd, lambda_rel, beta, warmup, stream=None):
        assert grads.dtype == self.grad_dtype and params.dtype == ema.dtype == torch.float32 and m.dtype == self.state_dtype
        rc = lib().adagc_step_lion(self._h, _ptr(params), _ptr(grads), _ptr(m), _ptr(ema), int(step), lr, beta1,
                                   beta2, wd, lambda_rel, beta, int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_lion")

    def step_sgdm(self, params, grads, m, ema, step, lr, momentum, wd, lambda_rel, beta, warmup, stream=None):
        assert grads.dtype == self.grad_dtype and params.dtype == ema.dtype == torch.float32 and m.dtype == self.state_dtype
        rc = lib().adagc_step_sgdm(self._h, _ptr(params), _ptr(grads), _ptr(m), _ptr(ema), int(step), lr, momentum,
                                   wd, lambda_rel, beta, int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_sgdm")

    def clip(self, grads_in, grads_out, ema, step, lambda_rel, beta, warmup, stream=None):
        assert grads_in.dtype == grads_out.dtype == self.grad_dtype and ema.dtype == torch.float32
        rc = lib().adagc_clip(self._h, _ptr(grads_in), _ptr(grads_out), _ptr(ema), int(step), lambda_rel, beta,
                              int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_clip")

    def step_host(self, params, grads_dev, m, v, ema, grads_host, step, lr, beta1, beta2, eps, wd, lambda_rel,
                  beta, warmup, norm_host=None, h_host=None, flag_host=None, stream=None):
        assert not grads_host.is_cuda and grads_host.dtype == self.grad_dtype
        rc = lib().adagc_step_host(self._h, _ptr(params), _ptr(grads_dev), _ptr(m), _ptr(v), _ptr(ema),
                                   _ptr(grads_host), int(step), lr, beta1, beta2, eps, wd, lambda_rel, beta,
                                   int(warmup), _ptr(norm_host), _ptr(h_host), _ptr(flag_host),
                                   _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_host")

    def shard_sumsq(self, grads, sumsq_out, stream=None):
        assert grads.dtype == self.grad_dtype and sumsq_out.dtype == torch.float64 and sumsq_out.is_cuda
        assert sumsq_out.numel() >= self.n_tensors and sumsq_out.is_contiguous()
        rc = lib().adagc_shard_sumsq(self._h, _ptr(grads), _ptr(sumsq_out), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_shard_sumsq")

    def step_presummed(self, params, grads, m, v, ema, sumsq, step, lr, beta1, beta2, eps, wd, lambda_rel, beta,
                       warmup, stream=None):
        assert grads.dtype == self.grad_dtype and params.dtype == ema.dtype == torch.float32 and m.dtype == v.dtype == self.state_dtype
        assert sumsq.dtype == torch.float64 and sumsq.is_cuda and sumsq.numel() >= self.n_tensors
        rc = lib().adagc_step_presummed(self._h, _ptr(params), _ptr(grads), _ptr(m), _ptr(v), _ptr(ema), _ptr(sumsq),
                                        int(step), lr, beta1, beta2, eps, wd, lambda_rel, beta, int(warmup),
                                        _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_step_presummed")

    def clip_presummed(self, grads_in, grads_out, ema, sumsq, step, lambda_rel, beta, warmup, stream=None):
        assert grads_in.dtype == grads_out.dtype == self.grad_dtype and ema.dtype == torch.float32
        assert sumsq.dtype == torch.float64 and sumsq.is_cuda and sumsq.numel() >= self.n_tensors
        rc = lib().adagc_clip_presummed(self._h, _ptr(grads_in), _ptr(grads_out), _ptr(ema), _ptr(sumsq), int(step),
                                        lambda_rel, beta, int(warmup), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_clip_presummed")

    def get_stats(self, stream=None):
        T = self.n_tensors
        norm, h = np.empty(T, np.float32), np.empty(T, np.float32)
        flag, cnt = np.empty(T, np.uint8), np.empty(T, np.uint64)
        steps, status = np.zeros(1, np.uint64), np.zeros(1, np.int32)
        rc = lib().adagc_get_stats(self._h, norm.ctypes.data, h.ctypes.data, flag.ctypes.data, cnt.ctypes.data,
                                   steps.ctypes.data, status.ctypes.data, _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_get_stats")
        return dict(norm=norm, h=h, flag=flag.astype(bool), clip_count=cnt, steps_done=int(steps[0]),
                    status=int(status[0]))

    def get_sumsq(self, stream=None) -> np.ndarray:
        out = np.empty(self.n_tensors, np.float64)
        rc = lib().adagc_get_sumsq(self._h, out.ctypes.data, _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_get_sumsq")
        return out

    def set_ema_cap(self, cap: float):
        rc = lib().adagc_set_ema_cap(self._h, float(cap))
        if rc != 0:
            raise AdagcError(rc, "adagc_set_ema_cap")

    def set_state_rounding(self, stochastic: bool, seed: int = 0):
        rc = lib().adagc_set_state_rounding(self._h, 1 if stochastic else 0, int(seed) & (2 ** 64 - 1))
        if rc != 0:
            raise AdagcError(rc, "adagc_set_state_rounding")

    def debug_wait_timeout(self, limit_ms: float, stream=None):
        rc = lib().adagc_debug_wait_timeout(self._h, float(limit_ms), _stream_ptr(stream))
        if rc != 0:
            raise AdagcError(rc, "adagc_debug_wait_timeout")

    def debug_latch_status(self, device_status: int):
        rc = lib().adagc_debug_latch_status(self._h, int(device_status))
        if rc != 0:
            raise AdagcError(rc, "adagc_debug_latch_status")

    def launch_count(self) -> int:
        return int(lib().adagc_launch_count(self._h))

    def launch_grids(self):
        """adagc_launch_grids: (blocks of the norm / scale kernels, blocks of the update kernel)."""
        n, u = C.c_int32(), C.c_int32()
        rc = lib().adagc_launch_grids(self._h, C.byref(n), C.byref(u))
        if rc != 0:
            raise AdagcError(rc, "adagc_launch_grids")
        return int(n.value), int(u.value)

    def set_phase_timing(self, enabled: bool):
        rc = lib().adagc_set_phase_timing(self._h, 1 if enabled else 0)
        if rc != 0:
            raise AdagcError(rc, "adagc_set_phase_timing")

    def get_phase_times(self):
        ms = (C.c_float * 3)()
        rc = lib().adagc_get_phase_times(self._h, ms)
        if rc != 0:
            raise AdagcError(rc, "adagc_get_phase_times")
        return [float(x) for x in ms]
