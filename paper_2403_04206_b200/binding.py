"""ctypes binding of libgrawa.so: argument marshalling only.

Each function has the name of the C entry point it calls (see ``include/grawa.h`` for the
meaning of every argument).  Device buffers are passed as torch CUDA tensors (float32,
contiguous, 1-D) or as raw integer device addresses; torch is used for device memory and
streams only.  Every step of the update runs in the library's CUDA kernels.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

import numpy as np

from . import build as _build

GRAWA_MAX_WORKERS = 64
_VARIANTS = {"grawa": 0, "mgrawa": 1, "lgrawa": 2}


class GrawaError(RuntimeError):
    """A libgrawa entry point returned a negative status."""

    def __init__(self, status: int, where: str):
        self.status = status
        text = library().grawa_status_string(status).decode()
        detail = library().grawa_last_cuda_error().decode() if status == -2 else ""
        super().__init__(f"{where}: {text} ({status})" + (f": {detail}" if detail else ""))


class _Options(ctypes.Structure):
    _fields_ = [("weights_out", ctypes.c_void_p), ("scores_out", ctypes.c_void_p), ("sumsq_out", ctypes.c_void_p),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t), ("status_word", ctypes.c_void_p)]


_lib = None


def library() -> ctypes.CDLL:
    """Loads (building first when missing or stale) libgrawa.so.  Raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    import os
    path = _build.build(debug_bounds=os.environ.get("GRAWA_DEBUG_BOUNDS", "0") == "1",
                        trace=os.environ.get("GRAWA_TRACE", "0") == "1")
    lib = ctypes.CDLL(path)
    vp, i64, ci, cf = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    step_args = [vp, vp, i64, ci, cf, vp, ci, vp, vp, vp]
    for name in ("grawa_mgrawa_step", "grawa_grawa_step", "grawa_lgrawa_step"):
        getattr(lib, name).argtypes = step_args
        getattr(lib, name).restype = ci
    lib.grawa_step_typed.argtypes = [ci, ci, vp, vp, i64, ci, cf, vp, ci, vp, vp, vp]
    lib.grawa_step_typed.restype = ci
    lib.grawa_step_host.argtypes = [ci, vp, vp, i64, ci, cf, vp, ci, vp, vp]
    lib.grawa_step_host.restype = ci
    lib.grawa_prox_step.argtypes = [vp, vp, i64, ci, cf, vp]
    lib.grawa_prox_step.restype = ci
    lib.grawa_workspace_bytes.argtypes = [i64, ci, vp, ci]
    lib.grawa_workspace_bytes.restype = ctypes.c_size_t
    lib.grawa_last_step_status.argtypes = [vp]
    lib.grawa_last_step_status.restype = ci
    lib.grawa_status_string.argtypes = [ci]
    lib.grawa_status_string.restype = ctypes.c_char_p
    lib.grawa_last_cuda_error.argtypes = []
    lib.grawa_last_cuda_error.restype = ctypes.c_char_p
    lib.grawa_version.restype = ci
    lib.grawa_set_option.argtypes = [ctypes.c_char_p, i64]
    lib.grawa_set_option.restype = ci
    lib.grawa_get_option.argtypes = [ctypes.c_char_p]
    lib.grawa_get_option.restype = i64
    lib.grawa_launch_count.restype = i64
    lib.grawa_clear_plans.restype = None
    lib.grawa_layer_norms.argtypes = [vp, i64, vp, ci, vp, vp]
    lib.grawa_layer_norms.restype = ci
    lib.grawa_norm_ema.argtypes = [vp, vp, ci, ctypes.c_double, i64, vp, vp]
    lib.grawa_norm_ema.restype = ci
    lib.grawa_step_from_layer_norms.argtypes = [ci, vp, vp, i64, ci, cf, vp, ci, vp, vp, vp]
    lib.grawa_step_from_layer_norms.restype = ci
    lib.grawa_layer_sumsq.argtypes = [vp, i64, ci, vp, ci, vp, vp]
    lib.grawa_layer_sumsq.restype = ci
    lib.grawa_step_from_layer_sums.argtypes = [ci, vp, vp, ci, i64, ci, cf, vp, ci, vp, vp, vp]
    lib.grawa_step_from_layer_sums.restype = ci
    lib.grawa_prox_step_typed.argtypes = [ci, vp, vp, i64, ci, cf, vp]
    lib.grawa_prox_step_typed.restype = ci
    lib.grawa_layer_norms_typed.argtypes = [ci, vp, i64, vp, ci, vp, vp]
    lib.grawa_layer_norms_typed.restype = ci
    lib.grawa_layer_sumsq_typed.argtypes = [ci, vp, i64, ci, vp, ci, vp, vp]
    lib.grawa_layer_sumsq_typed.restype = ci
    lib.grawa_step_from_layer_norms_typed.argtypes = [ci, ci, vp, vp, i64, ci, cf, vp, ci, vp, vp, vp]
    lib.grawa_step_from_layer_norms_typed.restype = ci
    lib.grawa_step_from_layer_sums_typed.argtypes = [ci, ci, vp, vp, ci, i64, ci, cf, vp, ci, vp, vp, vp]
    lib.grawa_step_from_layer_sums_typed.restype = ci
    lib.grawa_step_host_typed.argtypes = [ci, ci, vp, vp, i64, ci, cf, vp, ci, vp, vp]
    lib.grawa_step_host_typed.restype = ci
    lib.grawa_sumsq_static.argtypes = [vp, i64, ci, vp, vp]
    lib.grawa_sumsq_static.restype = ci
    lib.grawa_debug_bounds_violations.argtypes = [ci]
    lib.grawa_debug_bounds_violations.restype = i64
    lib.grawa_trace_read.argtypes = [vp, ci]
    lib.grawa_trace_read.restype = ci
    lib.grawa_selftest_bounded_wait.argtypes = [i64, vp]
    lib.grawa_selftest_bounded_wait.restype = ci
    lib.grawa_collect_kernel_times.argtypes = [vp, vp, vp, vp]
    lib.grawa_collect_kernel_times.restype = ci
    _lib = lib
    return lib


# ------------------------------------------------------------------ marshalling helpers

def _addr(buf) -> int:
    """Device (or host) address of a torch tensor / numpy array / integer / None."""
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if isinstance(buf, np.ndarray):
        if not buf.flags["C_CONTIGUOUS"]:
            raise ValueError("numpy buffers must be C-contiguous")
        return buf.ctypes.data
    if hasattr(buf, "data_ptr"):
        if not buf.is_contiguous():
            raise ValueError("tensors must be contiguous")
        return buf.data_ptr()
    raise TypeError(f"cannot take the address of {type(buf)!r}")


def _numel(buf) -> int:
    if isinstance(buf, np.ndarray):
        return buf.size
    return buf.numel()


def _check_f32(bufs):
    for b in bufs:
        if hasattr(b, "dtype") and str(b.dtype) not in ("torch.float32", "float32"):
            raise TypeError(f"expected float32 buffers, got {b.dtype}")


def _ptr_array(bufs: Sequence) -> ctypes.Array:
    return (ctypes.c_void_p * len(bufs))(*[_addr(b) for b in bufs])


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _offsets(layer_offsets):
    if layer_offsets is None:
        return None, 0
    off = np.ascontiguousarray(np.asarray(layer_offsets), dtype=np.int64)
    return off, off.size - 1


def _raise(status: int, where: str):
    if status < 0:
        raise GrawaError(status, where)


def _options(weights_out=None, scores_out=None, sumsq_out=None, workspace=None, status_word=None):
    """The optional-arguments struct, or None when every option is at its default."""
    if all(b is None for b in (weights_out, scores_out, sumsq_out, workspace, status_word)):
        return None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    return _Options(_addr(weights_out), _addr(scores_out), _addr(sumsq_out), _addr(workspace), ws_bytes, _addr(status_word))


def _byref(opt):
    return ctypes.byref(opt) if opt is not None else None


_DTYPES = {"torch.float32": 0, "torch.bfloat16": 1, "torch.float16": 2, "float32": 0, "float16": 2}


def _dtype_of(bufs) -> int:
    """Storage type code of a list of buffers (all of one type)."""
    key = str(bufs[0].dtype)
    if key not in _DTYPES:
        raise TypeError(f"unsupported storage dtype {key}")
    for b in bufs:
        if str(b.dtype) != key:
            raise TypeError(f"all buffers must be {key}, got {b.dtype}")
    return _DTYPES[key]


def _step(name, params, grads, pull, layer_offsets, center_out, weights_out, scores_out, sumsq_out,
          workspace, stream, n, status_word=None):
    lib = library()
    if len(params) != len(grads):
        raise ValueError("params and grads must have one entry per worker")
    _check_f32(list(params) + list(grads) + ([center_out] if center_out is not None else []))
    M = len(params)
    if n is None:
        n = _numel(params[0]) if M else 0
    off, K = _offsets(layer_offsets)
    opt = _options(weights_out, scores_out, sumsq_out, workspace, status_word)
    status = getattr(lib, name)(_ptr_array(params), _ptr_array(grads), n, M, float(pull),
                                off.ctypes.data if off is not None else None, K, _addr(center_out),
                                _byref(opt), _stream(stream))
    _raise(status, name)


# ------------------------------------------------------------------ entry points (same names as the C ABI)

def grawa_mgrawa_step(params, grads, pull, layer_offsets=None, center_out=None, *, weights_out=None,
                      scores_out=None, sumsq_out=None, workspace=None, stream=None, n=None, status_word=None) -> None:
    """MGRAWA step (Eq. 3-4, centre, pull) in place on ``params``; see grawa_mgrawa_step in grawa.h."""
    _step("grawa_mgrawa_step", params, grads, pull, layer_offsets, center_out, weights_out, scores_out,
          sumsq_out, workspace, stream, n, status_word)


def grawa_grawa_step(params, grads, pull, layer_offsets=None, center_out=None, *, weights_out=None,
                     scores_out=None, sumsq_out=None, workspace=None, stream=None, n=None, status_word=None) -> None:
    """Vanilla GRAWA step (Eq. 2: flat gradient norm); see grawa_grawa_step in grawa.h."""
    _step("grawa_grawa_step", params, grads, pull, layer_offsets, center_out, weights_out, scores_out,
          sumsq_out, workspace, stream, n, status_word)


def grawa_lgrawa_step(params, grads, pull, layer_offsets, center_out=None, *, weights_out=None,
                      scores_out=None, sumsq_out=None, workspace=None, stream=None, n=None, status_word=None) -> None:
    """LGRAWA step (Eq. 5-7: per-layer weights); see grawa_lgrawa_step in grawa.h."""
    _step("grawa_lgrawa_step", params, grads, pull, layer_offsets, center_out, weights_out, scores_out,
          sumsq_out, workspace, stream, n, status_word)


def grawa_step_typed(variant, params, grads, pull, layer_offsets=None, center_out=None, *, weights_out=None,
                     scores_out=None, sumsq_out=None, workspace=None, stream=None, n=None, status_word=None) -> None:
    """The step on parameters / gradients / centre stored as float32, bfloat16 or float16 device tensors
    (all of one dtype, taken from ``params[0]``); arithmetic in fp32/fp64, one rounding per stored value."""
    M = len(params)
    if len(grads) != M or M == 0:
        raise ValueError("params and grads must have one entry per worker")
    dt = _dtype_of(list(params) + list(grads) + ([center_out] if center_out is not None else []))
    v = _VARIANTS[variant] if isinstance(variant, str) else int(variant)
    if n is None:
        n = _numel(params[0])
    off, K = _offsets(layer_offsets)
    opt = _options(weights_out, scores_out, sumsq_out, workspace, status_word)
    _raise(library().grawa_step_typed(dt, v, _ptr_array(params), _ptr_array(grads), n, M, float(pull),
                                      off.ctypes.data if off is not None else None, K, _addr(center_out),
                                      _byref(opt), _stream(stream)), "grawa_step_typed")


def grawa_step_host_typed(variant, params, grads, pull, layer_offsets=None, center_out=None, *, stream=None, n=None) -> None:
    """Whole step with HOST buffers (numpy arrays or pinned CPU tensors) of float32, float16 or bfloat16;
    synchronises before returning."""
    v = _VARIANTS[variant] if isinstance(variant, str) else int(variant)
    M = len(params)
    dt = _dtype_of(list(params) + list(grads) + ([center_out] if center_out is not None else []))
    if n is None:
        n = _numel(params[0]) if M else 0
    off, K = _offsets(layer_offsets)
    _raise(library().grawa_step_host_typed(dt, v, _ptr_array(params), _ptr_array(grads), n, M, float(pull),
                                           off.ctypes.data if off is not None else None, K, _addr(center_out),
                                           _stream(stream)), "grawa_step_host_typed")


def grawa_step_host(variant, params, grads, pull, layer_offsets=None, center_out=None, *, stream=None, n=None) -> None:
    """Whole step with HOST float32 buffers (numpy arrays or pinned CPU tensors); synchronises before returning."""
    lib = library()
    v = _VARIANTS[variant] if isinstance(variant, str) else int(variant)
    _check_f32(list(params) + list(grads) + ([center_out] if center_out is not None else []))
    M = len(params)
    if n is None:
        n = _numel(params[0]) if M else 0
    off, K = _offsets(layer_offsets)
    status = lib.grawa_step_host(v, _ptr_array(params), _ptr_array(grads), n, M, float(pull),
                                 off.ctypes.data if off is not None else None, K, _addr(center_out), _stream(stream))
    _raise(status, "grawa_step_host")


def grawa_prox_step_typed(params, center, mu_over_tau, *, stream=None, n=None) -> None:
    """Proximity step on float32, bfloat16 or float16 device tensors (dtype taken from the buffers)."""
    dt = _dtype_of(list(params) + [center])
    if n is None:
        n = _numel(center)
    _raise(library().grawa_prox_step_typed(dt, _ptr_array(params), _addr(center), n, len(params), float(mu_over_tau),
                                           _stream(stream)), "grawa_prox_step_typed")


def grawa_prox_step(params, center, mu_over_tau, *, stream=None, n=None) -> None:
    """Proximity step x_m <- (1 - mu/tau) x_m + (mu/tau) x_C for all workers in one pass."""
    lib = library()
    _check_f32(list(params) + [center])
    M = len(params)
    if n is None:
        n = _numel(center)
    _raise(lib.grawa_prox_step(_ptr_array(params), _addr(center), n, M, float(mu_over_tau), _stream(stream)),
           "grawa_prox_step")


def grawa_layer_norms_typed(grad, layer_offsets, norms_out, *, stream=None, n=None) -> None:
    """Per-layer L2 norms of one worker's gradient (float32, bfloat16 or float16) into ``norms_out`` (K float64)."""
    dt = _dtype_of([grad])
    if n is None:
        n = _numel(grad)
    off, K = _offsets(layer_offsets)
    _raise(library().grawa_layer_norms_typed(dt, _addr(grad), n, off.ctypes.data if off is not None else None, K,
                                             _addr(norms_out), _stream(stream)), "grawa_layer_norms_typed")


def grawa_layer_norms(grad, layer_offsets, norms_out, *, stream=None, n=None) -> None:
    """Per-layer L2 norms of one worker's gradient into ``norms_out`` (device, K float64)."""
    _check_f32([grad])
    if n is None:
        n = _numel(grad)
    off, K = _offsets(layer_offsets)
    _raise(library().grawa_layer_norms(_addr(grad), n, off.ctypes.data if off is not None else None, K,
                                       _addr(norms_out), _stream(stream)), "grawa_layer_norms")


def grawa_norm_ema(g_mvg, g_cur, gamma, t, g_est, *, stream=None) -> None:
    """Running norm estimate of the Local variants on device float64 vectors (g_mvg updated in place)."""
    _raise(library().grawa_norm_ema(_addr(g_mvg), _addr(g_cur), _numel(g_mvg), float(gamma), int(t), _addr(g_est),
                                    _stream(stream)), "grawa_norm_ema")


def _from_given(name, typed, variant, params, table, parts, pull, layer_offsets, center_out, weights_out, scores_out,
                sumsq_out, workspace, stream, n, status_word):
    v = _VARIANTS[variant] if isinstance(variant, str) else int(variant)
    bufs = list(params) + ([center_out] if center_out is not None else [])
    M = len(params)
    if n is None:
        n = _numel(params[0]) if M else 0
    off, K = _offsets(layer_offsets)
    opt = _options(weights_out, scores_out, sumsq_out, workspace, status_word)
    head = [_dtype_of(bufs), v] if typed else [v]
    if not typed:
        _check_f32(bufs)
    mid = [_ptr_array(params), _addr(table)] + ([int(parts)] if parts is not None else [])
    tail = [n, M, float(pull), off.ctypes.data if off is not None else None, K, _addr(center_out), _byref(opt), _stream(stream)]
    _raise(getattr(library(), name)(*(head + mid + tail)), name)


def grawa_step_from_layer_norms(variant, params, layer_norms, pull, layer_offsets=None, center_out=None, *,
                                weights_out=None, scores_out=None, sumsq_out=None, workspace=None, stream=None,
                                n=None, status_word=None) -> None:
    """Averaging step with scores from given per-layer norms ([K, M] device float64) instead of gradients."""
    _from_given("grawa_step_from_layer_norms", False, variant, params, layer_norms, None, pull, layer_offsets, center_out,
                weights_out, scores_out, sumsq_out, workspace, stream, n, status_word)


def grawa_step_from_layer_norms_typed(variant, params, layer_norms, pull, layer_offsets=None, center_out=None, *,
                                      weights_out=None, scores_out=None, sumsq_out=None, workspace=None, stream=None,
                                      n=None, status_word=None) -> None:
    """The same on float32, bfloat16 or float16 parameters and centre."""
    _from_given("grawa_step_from_layer_norms_typed", True, variant, params, layer_norms, None, pull, layer_offsets,
                center_out, weights_out, scores_out, sumsq_out, workspace, stream, n, status_word)


def grawa_layer_sumsq(grads, layer_offsets, sumsq_out, *, stream=None, n=None) -> None:
    """Per-layer sums of squares of the M workers' local gradients into ``sumsq_out`` ([K, M] device float64)."""
    _check_f32(list(grads))
    M = len(grads)
    if n is None:
        n = _numel(grads[0]) if M else 0
    off, K = _offsets(layer_offsets)
    _raise(library().grawa_layer_sumsq(_ptr_array(grads), n, M, off.ctypes.data if off is not None else None, K,
                                       _addr(sumsq_out), _stream(stream)), "grawa_layer_sumsq")


def grawa_layer_sumsq_typed(grads, layer_offsets, sumsq_out, *, stream=None, n=None) -> None:
    """The same from float32, bfloat16 or float16 gradients."""
    M = len(grads)
    dt = _dtype_of(list(grads))
    if n is None:
        n = _numel(grads[0]) if M else 0
    off, K = _offsets(layer_offsets)
    _raise(library().grawa_layer_sumsq_typed(dt, _ptr_array(grads), n, M, off.ctypes.data if off is not None else None, K,
                                             _addr(sumsq_out), _stream(stream)), "grawa_layer_sumsq_typed")


def grawa_step_from_layer_sums(variant, params, layer_sums, parts, pull, layer_offsets=None, center_out=None, *,
                               weights_out=None, scores_out=None, sumsq_out=None, workspace=None, stream=None,
                               n=None, status_word=None) -> None:
    """Averaging step on local elements with S = sum over ``parts`` tables of ``layer_sums`` ([parts, K, M])."""
    _from_given("grawa_step_from_layer_sums", False, variant, params, layer_sums, parts, pull, layer_offsets, center_out,
                weights_out, scores_out, sumsq_out, workspace, stream, n, status_word)


def grawa_step_from_layer_sums_typed(variant, params, layer_sums, parts, pull, layer_offsets=None, center_out=None, *,
                                     weights_out=None, scores_out=None, sumsq_out=None, workspace=None, stream=None,
                                     n=None, status_word=None) -> None:
    """The same on float32, bfloat16 or float16 parameters and centre."""
    _from_given("grawa_step_from_layer_sums_typed", True, variant, params, layer_sums, parts, pull, layer_offsets,
                center_out, weights_out, scores_out, sumsq_out, workspace, stream, n, status_word)


class PreparedStep:
    """A device-buffer step with its arguments marshalled once: calling the object makes the same C call
    (grawa_step_typed) again on the stream that is current at that moment.  For loops over small models,
    where building the pointer tables in Python costs as much as the update.  Holds references to the
    buffers; marshals only, like every function of this module."""

    def __init__(self, variant, params, grads, pull, layer_offsets=None, center_out=None, *, status_word=None):
        self._keep = (list(params), list(grads), center_out, status_word)
        self._dt = _dtype_of(list(params) + list(grads) + ([center_out] if center_out is not None else []))
        self._v = _VARIANTS[variant] if isinstance(variant, str) else int(variant)
        self._params, self._grads = _ptr_array(params), _ptr_array(grads)
        self._n, self._M, self._pull = _numel(params[0]), len(params), float(pull)
        self._off, self._K = _offsets(layer_offsets)
        self._off_ptr = self._off.ctypes.data if self._off is not None else None
        self._center = _addr(center_out)
        self._opt = _options(status_word=status_word)
        self._fn = library().grawa_step_typed

    def __call__(self, stream=None) -> None:
        status = self._fn(self._dt, self._v, self._params, self._grads, self._n, self._M, self._pull, self._off_ptr, self._K,
                          self._center, _byref(self._opt), _stream(stream))
        if status < 0:
            raise GrawaError(status, "grawa_step_typed")


def grawa_sumsq_static(grads, sumsq_out, *, stream=None, n=None) -> None:
    """Squared gradient norms of the M workers into ``sumsq_out`` (device, M float64) using only
    the scratch array built into the library: for callers whose device memory belongs to another
    allocator, or who cannot afford the synchronisation an allocation implies.  Calls that may
    overlap on the GPU share that array and race; keep them on one stream."""
    _check_f32(list(grads))
    M = len(grads)
    if n is None:
        n = _numel(grads[0]) if M else 0
    _raise(library().grawa_sumsq_static(_ptr_array(grads), n, M, _addr(sumsq_out), _stream(stream)),
           "grawa_sumsq_static")


def grawa_workspace_bytes(n: int, M: int, layer_offsets=None) -> int:
    off, K = _offsets(layer_offsets)
    return int(library().grawa_workspace_bytes(n, M, off.ctypes.data if off is not None else None, K))


def grawa_last_step_status(stream=None) -> int:
    """Synchronises the stream and returns the status code of the last step enqueued on it."""
    return int(library().grawa_last_step_status(_stream(stream)))


def grawa_status_string(status: int) -> str:
    return library().grawa_status_string(int(status)).decode()


def grawa_last_cuda_error() -> str:
    return library().grawa_last_cuda_error().decode()


def grawa_version() -> int:
    return int(library().grawa_version())


def grawa_set_option(name: str, value: int) -> None:
    _raise(library().grawa_set_option(name.encode(), int(value)), f"grawa_set_option({name})")


def grawa_get_option(name: str) -> int:
    return int(library().grawa_get_option(name.encode()))


def grawa_launch_count() -> int:
    return int(library().grawa_launch_count())


def grawa_collect_kernel_times() -> dict:
    """Per-phase device time (ms, summed) of the steps run while option "kernel_timing" was 1."""
    a, b, c = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    k = ctypes.c_int64()
    _raise(library().grawa_collect_kernel_times(ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(k)),
           "grawa_collect_kernel_times")
    return {"sumsq_ms": a.value, "finalize_ms": b.value, "center_pull_ms": c.value, "steps": k.value}


def grawa_selftest_bounded_wait(limit_ns: int, *, stream=None) -> None:
    """Launches the bounded-wait self-test; read the outcome with grawa_last_step_status (expect -5)."""
    _raise(library().grawa_selftest_bounded_wait(int(limit_ns), _stream(stream)), "grawa_selftest_bounded_wait")


def grawa_debug_bounds_violations(selfcheck: bool = False) -> int:
    """Violations counted by a bounds-checking debug build since the last call (-1 in a normal build)."""
    return int(library().grawa_debug_bounds_violations(1 if selfcheck else 0))


def grawa_trace_read(max_rows: int = 64):
    """Trace build (GRAWA_TRACE=1 in the environment): the rows stamped since the last call as an
    array [rows, 3 kernels, 4 stamps] of uint64 nanoseconds, and a reset.  None in the normal build."""
    buf = np.zeros((max_rows, 3, 4), dtype=np.uint64)
    kept = int(library().grawa_trace_read(buf.ctypes.data, max_rows))
    if kept == -1:
        return None
    if kept < 0:
        raise GrawaError(-2, "grawa_trace_read")
    return buf


def grawa_clear_plans() -> None:
    library().grawa_clear_plans()
