"""ctypes binding of the C-ABI library declared in ``include/came_b200.h``.

Argument marshalling only: every step of the optimizer runs in the CUDA
kernels of ``libcame_b200.so``.  The functions carry the C names
(``came_create``, ``came_step``, ...).  ``CameOptimizer`` is a small convenience
wrapper that owns the state tensors (allocated with torch) and a context.

There is no fallback: if the library is missing it is built with nvcc, and if
that fails, or a call returns an error status, a ``CameError`` is raised.
"""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence

from . import build as _build

CAME_OK = 0
CAME_F32, CAME_BF16 = 0, 1
CAME_T_NO_WEIGHT_DECAY = 1
CAME_T_VEC_NO_CONFIDENCE = 2
CAME_CREATE_KEEP_STATE = 1
CAME_CREATE_ADAFACTOR = 2
(CAME_Q_NUMEL, CAME_Q_STATE_BYTES, CAME_Q_STREAM_BYTES, CAME_Q_COMPULSORY_BYTES,
 CAME_Q_WORKSPACE_BYTES, CAME_Q_NUM_TILES, CAME_Q_LAUNCHES_PER_STEP, CAME_Q_LAST_STEP,
 CAME_Q_NUM_PHASES, CAME_Q_MATRIX_NUMEL, CAME_Q_SCHEDULE, CAME_Q_PIPE_GROUPS, CAME_Q_PIPE_GRID,
 CAME_Q_DEVICE_ERROR) = range(14)
CAME_Q_P1_STREAM_GRID = 14
CAME_TUNE_TILE_ELEMS = 0
CAME_TUNE_SCHED_GROUP_BYTES = 1
CAME_TUNE_HOST_GROUP_BYTES = 2
CAME_TUNE_PDL = 3
CAME_TUNE_F32_VEC8 = 4
CAME_TUNE_SCHEDULE = 5
CAME_TUNE_PIPE_TILE_ELEMS = 6
CAME_TUNE_PIPE_GROUP_BYTES = 7
CAME_TUNE_PIPE_WAIT_NS = 8
CAME_TUNE_PIPE_ORDER = 9
CAME_TUNE_P1_STREAM = 10
CAME_TUNE_P1_STREAM_RING = 11
CAME_SCHEDULE_AUTO, CAME_SCHEDULE_PHASE_GRIDS, CAME_SCHEDULE_PIPELINED = 0, 1, 2

EXPORTED = ["came_create", "came_step", "came_step_host", "came_destroy", "came_last_error",
            "came_status_string", "came_query", "came_set_profiling", "came_get_phase_ms",
            "came_phase_name", "came_plan_tensor", "came_tune", "came_factor_update_static",
            "came_factor_update_static_plan", "came_required_grad_alignment",
            "came_device_status", "came_lr_warmup", "came_clear_device_error",
            "came_selftest_wait_timeout", "came_debug_bounds"]


class CameError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{text} (status {status})")
        self.status = status


class came_tensor(ctypes.Structure):
    _fields_ = [("param", ctypes.c_void_p), ("grad", ctypes.c_void_p), ("m", ctypes.c_void_p),
                ("r", ctypes.c_void_p), ("c", ctypes.c_void_p), ("R", ctypes.c_void_p),
                ("C", ctypes.c_void_p), ("rows", ctypes.c_int64), ("cols", ctypes.c_int64),
                ("ndim", ctypes.c_int32), ("grad_dtype", ctypes.c_int32),
                ("flags", ctypes.c_uint32), ("reserved", ctypes.c_uint32),
                ("param_bf16", ctypes.c_void_p)]


class came_hparams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("beta3", ctypes.c_double), ("eps1", ctypes.c_double), ("eps2", ctypes.c_double),
                ("clip_d", ctypes.c_double), ("weight_decay", ctypes.c_double),
                ("step", ctypes.c_int64), ("grad_scale", ctypes.c_double)]


_lib = None


def load():
    """Load (building first if needed) the shared library; raises if it cannot be had."""
    global _lib
    if _lib is not None:
        return _lib
    _lib = _bind(ctypes.CDLL(_build.build()))
    return _lib


_lib_debug = None


def load_debug():
    """The bounds-checking build of the same library (``-DCAME_DEBUG_BOUNDS``), built on demand."""
    global _lib_debug
    if _lib_debug is None:
        _lib_debug = _bind(ctypes.CDLL(_build.build(debug=True)))
    return _lib_debug


class using_debug_build:
    """``with using_debug_build():`` routes every call of this module through the
    bounds-checking build for the duration of the block."""

    def __enter__(self):
        global _lib
        load()
        self.saved = _lib
        _lib = load_debug()
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved


def _bind(L):
    """Declare the prototypes of every entry point on a freshly loaded library."""
    vp, i32, i64, u32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32
    L.came_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(came_tensor), i32, i32, u32]
    L.came_create.restype = i32
    L.came_step.argtypes = [vp, ctypes.POINTER(came_hparams), ctypes.POINTER(vp), vp]
    L.came_step.restype = i32
    L.came_step_host.argtypes = [vp, ctypes.POINTER(came_hparams), ctypes.POINTER(vp),
                                 ctypes.POINTER(vp), vp]
    L.came_step_host.restype = i32
    L.came_destroy.argtypes = [vp]
    L.came_destroy.restype = i32
    L.came_last_error.argtypes = [vp]
    L.came_last_error.restype = ctypes.c_char_p
    L.came_status_string.argtypes = [i32]
    L.came_status_string.restype = ctypes.c_char_p
    L.came_query.argtypes = [vp, i32, ctypes.POINTER(i64)]
    L.came_query.restype = i32
    L.came_set_profiling.argtypes = [vp, i32]
    L.came_set_profiling.restype = i32
    L.came_get_phase_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float), i32, ctypes.POINTER(i32)]
    L.came_get_phase_ms.restype = i32
    L.came_phase_name.argtypes = [vp, i32]
    L.came_phase_name.restype = ctypes.c_char_p
    L.came_plan_tensor.argtypes = [i64, i64, i32, i32, i32, i64] + [ctypes.POINTER(i32)] * 5
    L.came_plan_tensor.restype = i32
    L.came_tune.argtypes = [i32, i64]
    L.came_tune.restype = i32
    L.came_factor_update_static.argtypes = [vp, i32, i64, i64, vp, vp, ctypes.c_double,
                                            ctypes.c_double, vp, i32, vp]
    L.came_factor_update_static.restype = i32
    L.came_factor_update_static_plan.argtypes = [vp, i32, i64, i64, vp, vp, ctypes.c_double,
                                                 ctypes.c_double, i32, ctypes.POINTER(i32),
                                                 ctypes.POINTER(i64)]
    L.came_factor_update_static_plan.restype = i32
    L.came_required_grad_alignment.argtypes = [i32, i32]
    L.came_required_grad_alignment.restype = i32
    L.came_device_status.argtypes = [i32, i32]
    L.came_device_status.restype = i32
    L.came_lr_warmup.argtypes = [ctypes.c_double, ctypes.c_double, i64, i64]
    L.came_lr_warmup.restype = ctypes.c_double
    L.came_clear_device_error.argtypes = [vp, vp]
    L.came_clear_device_error.restype = i32
    L.came_selftest_wait_timeout.argtypes = [i32, i64, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                             ctypes.POINTER(ctypes.c_float)]
    L.came_selftest_wait_timeout.restype = i32
    L.came_debug_bounds.argtypes = [i32, ctypes.POINTER(ctypes.c_uint32)]
    L.came_debug_bounds.restype = i32
    return L


def _check(status: int, ctx=None) -> None:
    if status != CAME_OK:
        L = load()
        text = L.came_last_error(ctx).decode() or L.came_status_string(status).decode()
        raise CameError(status, f"{L.came_status_string(status).decode()}: {text}")


# --- the C entry points, same names ------------------------------------------------------

def came_create(tensors: Sequence[came_tensor], device: int = 0, flags: int = 0) -> ctypes.c_void_p:
    L = load()
    arr = (came_tensor * len(tensors))(*tensors)
    ctx = ctypes.c_void_p()
    _check(L.came_create(ctypes.byref(ctx), arr, len(tensors), device, flags))
    return ctx


def came_step(ctx, hp: came_hparams, grads: Optional[Sequence[int]] = None, stream: int = 0) -> None:
    L = load()
    garr = None
    if grads is not None:
        garr = (ctypes.c_void_p * len(grads))(*grads)
    _check(L.came_step(ctx, ctypes.byref(hp), garr, ctypes.c_void_p(stream)), ctx)


def came_step_host(ctx, hp: came_hparams, host_grads: Sequence[int],
                   host_params_out: Optional[Sequence[Optional[int]]] = None, stream: int = 0) -> None:
    L = load()
    garr = (ctypes.c_void_p * len(host_grads))(*host_grads)
    parr = None
    if host_params_out is not None:
        parr = (ctypes.c_void_p * len(host_params_out))(*host_params_out)
    _check(L.came_step_host(ctx, ctypes.byref(hp), garr, parr, ctypes.c_void_p(stream)), ctx)


def came_destroy(ctx) -> None:
    _check(load().came_destroy(ctx))


def came_last_error(ctx=None) -> str:
    return load().came_last_error(ctx).decode()


def came_status_string(status: int) -> str:
    return load().came_status_string(status).decode()


def came_query(ctx, what: int) -> int:
    out = ctypes.c_int64()
    _check(load().came_query(ctx, what, ctypes.byref(out)), ctx)
    return int(out.value)


def came_set_profiling(ctx, enabled: bool) -> None:
    _check(load().came_set_profiling(ctx, int(enabled)), ctx)


def came_get_phase_ms(ctx) -> List[float]:
    buf = (ctypes.c_float * 8)()
    cnt = ctypes.c_int32()
    _check(load().came_get_phase_ms(ctx, buf, 8, ctypes.byref(cnt)), ctx)
    return [float(buf[i]) for i in range(cnt.value)]


def came_phase_name(ctx, phase: int) -> str:
    return load().came_phase_name(ctx, phase).decode()


def came_plan_tensor(rows: int, cols: int, ndim: int, grad_dtype: int, aligned32: bool = True,
                     tile_elems_target: int = 0) -> dict:
    o = [ctypes.c_int32() for _ in range(5)]
    _check(load().came_plan_tensor(rows, cols, ndim, grad_dtype, int(aligned32), tile_elems_target,
                                   *[ctypes.byref(x) for x in o]))
    return dict(zip(("vec", "threads_x", "tile_rows", "n_rb", "n_cb"), (int(x.value) for x in o)))


def came_tune(key: int, value: int) -> None:
    _check(load().came_tune(key, value))


CAME_STATIC_SCRATCH_BYTES = 8 << 20


def came_factor_update_static(grad: int, grad_dtype: int, rows: int, cols: int, r: int, c: int,
                              beta2: float, eps1: float, out_sqrt_sum_r: Optional[int] = None,
                              device: int = 0, stream: int = 0) -> None:
    """r, c <- the first two lines of Algorithm 2 for one matrix, without any allocation.

    For callers that may not allocate device memory (an allocator that owns the device
    heap, a no-synchronisation loop, an audited memory budget): the partial sums use a
    fixed array inside the library instead of a context's workspace.  All pointer
    arguments are device addresses (ints).  Calls share that array: keep them on one stream.
    """
    _check(load().came_factor_update_static(grad, grad_dtype, rows, cols, r, c, float(beta2),
                                            float(eps1), out_sqrt_sum_r, device,
                                            ctypes.c_void_p(stream)))


def came_factor_update_static_plan(grad: int, grad_dtype: int, rows: int, cols: int, r: int, c: int,
                                   beta2: float = 0.999, eps1: float = 1e-30, device: int = 0) -> dict:
    """Host-only: what came_factor_update_static would plan for these arguments (no GPU work)."""
    vec, nbytes = ctypes.c_int32(), ctypes.c_int64()
    _check(load().came_factor_update_static_plan(grad, grad_dtype, rows, cols, r, c, float(beta2),
                                                 float(eps1), device, ctypes.byref(vec),
                                                 ctypes.byref(nbytes)))
    return {"vec": int(vec.value), "scratch_bytes": int(nbytes.value)}


def came_required_grad_alignment(grad_dtype: int, vec: int) -> int:
    return int(load().came_required_grad_alignment(grad_dtype, vec))


def came_device_status(context_device: int, current_device: int) -> int:
    return int(load().came_device_status(context_device, current_device))


def came_lr_warmup(lr_peak: float, lr_start: float, step: int, warmup_steps: int) -> float:
    return float(load().came_lr_warmup(lr_peak, lr_start, step, warmup_steps))


def came_clear_device_error(ctx, stream: int = 0) -> None:
    _check(load().came_clear_device_error(ctx, ctypes.c_void_p(stream)), ctx)


def came_selftest_wait_timeout(device: int = 0, limit_ns: int = 1_000_000) -> dict:
    a, b, ms = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_float()
    _check(load().came_selftest_wait_timeout(device, limit_ns, ctypes.byref(a), ctypes.byref(b),
                                             ctypes.byref(ms)))
    return {"timed_out": int(a.value), "error_word": int(b.value), "elapsed_ms": float(ms.value)}


def came_debug_bounds(device: int = 0) -> dict:
    """The device-side record of the bounds-checking build (raises CAME_ERR_UNSUPPORTED, status
    11, on the ordinary build)."""
    out = (ctypes.c_uint32 * 6)()
    _check(load().came_debug_bounds(device, out))
    return dict(zip(("code", "rb", "cb", "rows", "cols", "threads"), (int(x) for x in out)))


def make_hparams(step: int, **kw) -> came_hparams:
    return came_hparams(float(kw["lr"]), float(kw["beta1"]), float(kw["beta2"]), float(kw["beta3"]),
                        float(kw["eps1"]), float(kw["eps2"]), float(kw["clip_d"]),
                        float(kw.get("weight_decay", 0.0)), int(step),
                        float(kw.get("grad_scale", 1.0)))


# --- convenience wrapper -------------------------------------------------------------------

class CameOptimizer:
    """Owns the CAME state for a list of torch CUDA parameter tensors and steps them.

    ``params``: fp32 CUDA tensors (contiguous), updated in place.  1-D tensors take the vector
    path, 2-D tensors the matrix path; a tensor of rank >= 3 is handed to the library as the
    matrix (product of the leading dims) x (last dim), since the paper defines the method for
    matrices only.
    ``grads``: CUDA tensors of the same shapes, fp32 or bf16, read every step
    (their storage may be refilled between steps; pointers are fixed at creation).
    torch is used for allocation and the stream only.
    """

    def __init__(self, params, grads, flags: Optional[Sequence[int]] = None, device: int = 0,
                 create_flags: int = 0, bf16_copy: bool = False):
        import torch
        self.torch = torch
        self.params, self.grads = list(params), list(grads)
        self.m, self.r, self.c, self.R, self.C = [], [], [], [], []
        self.p_bf16 = []
        descs = []
        for i, (p, g) in enumerate(zip(self.params, self.grads)):
            assert p.is_cuda and p.dtype == torch.float32 and p.is_contiguous()
            assert g.is_cuda and g.is_contiguous() and g.shape == p.shape
            assert p.dim() >= 1
            ndim = 1 if p.dim() == 1 else 2
            cols = p.shape[-1] if ndim == 2 else 1
            rows = p.numel() // cols
            z = lambda n: torch.empty(n, dtype=torch.float32, device=p.device)
            self.m.append(torch.empty_like(p))
            self.r.append(z(rows)); self.R.append(z(rows))
            self.c.append(z(cols) if ndim == 2 else None)
            self.C.append(z(cols) if ndim == 2 else None)
            gd = CAME_BF16 if g.dtype == torch.bfloat16 else CAME_F32
            assert g.dtype in (torch.bfloat16, torch.float32)
            ptr = lambda t: t.data_ptr() if t is not None else None
            self.p_bf16.append(torch.empty_like(p, dtype=torch.bfloat16) if bf16_copy else None)
            descs.append(came_tensor(ptr(p), ptr(g), ptr(self.m[i]), ptr(self.r[i]), ptr(self.c[i]),
                                     ptr(self.R[i]), ptr(self.C[i]), rows, cols, ndim, gd,
                                     0 if flags is None else int(flags[i]), 0, ptr(self.p_bf16[i])))
        self.ctx = came_create(descs, device=device, flags=create_flags)
        self.step_count = 0

    def step(self, **hp) -> None:
        self.step_count += 1
        stream = self.torch.cuda.current_stream().cuda_stream
        came_step(self.ctx, make_hparams(self.step_count, **hp), None, stream)

    def query(self, what: int) -> int:
        return came_query(self.ctx, what)

    def close(self) -> None:
        if self.ctx is not None:
            self.torch.cuda.synchronize()
            came_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
