"""Thin ctypes binding over the C ABI declared in ``include/patdnn.h``.

Argument marshalling only: every step of the path (encode, reorder, launch) runs inside ``libpatdnn.so``.  Device
buffers are passed as raw pointers (``tensor.data_ptr()`` of a torch CUDA tensor, or any integer address); host
buffers as numpy arrays.  There is no CPU fallback: if the shared library is missing, loading fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libpatdnn.so")

OK = 0
F32, F16 = 0, 1
VARIANT_AUTO, VARIANT_NOOPT, VARIANT_REORDER, VARIANT_TILED, VARIANT_DENSE_TC, VARIANT_PATTERN_RUN = 0, 1, 2, 3, 4, 5
FLAG_HOST_ONLY = 1
STATUS_NAMES = {0: "OK", 1: "E_NULL", 2: "E_SHAPE", 3: "E_PATTERN_SET", 4: "E_MASK", 5: "E_ORDER", 6: "E_CUDA",
                7: "E_NO_DEVICE", 8: "E_DEVICE_TIMEOUT", 9: "E_DTYPE", 10: "E_ALLOC", 11: "E_STACK", 12: "E_SCRATCH"}

EXPORTED_SYMBOLS = (
    "patdnn_encode", "patdnn_conv", "patdnn_conv_static", "patdnn_conv_host", "patdnn_check", "patdnn_free", "patdnn_export", "patdnn_decode",
    "patdnn_plan", "patdnn_stack_create", "patdnn_stack_run", "patdnn_stack_run_host", "patdnn_stack_out_shape",
    "patdnn_stack_free", "patdnn_stack_submit_host", "patdnn_stack_wait_host", "patdnn_maxpool2x2", "patdnn_launch_count", "patdnn_reset_launch_count", "patdnn_strerror",
    "patdnn_last_cuda_error", "patdnn_version", "patdnn_debug_wait", "patdnn_stack_run_timed", "patdnn_stack_generated",
)


class PatdnnError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({detail})")


class _Desc(ctypes.Structure):
    _fields_ = [("F", ctypes.c_int32), ("C", ctypes.c_int32), ("N", ctypes.c_int32), ("H", ctypes.c_int32),
                ("W", ctypes.c_int32), ("dtype", ctypes.c_int32), ("relu", ctypes.c_int32),
                ("filter_order", ctypes.c_int32), ("order", ctypes.POINTER(ctypes.c_int32)),
                ("bias", ctypes.POINTER(ctypes.c_float)), ("variant", ctypes.c_int32), ("flags", ctypes.c_int32)]


class _FkwView(ctypes.Structure):
    _fields_ = [("F", ctypes.c_int32), ("C", ctypes.c_int32), ("P", ctypes.c_int32), ("K", ctypes.c_int32),
                ("offset", ctypes.POINTER(ctypes.c_int32)), ("reorder", ctypes.POINTER(ctypes.c_int32)),
                ("index", ctypes.POINTER(ctypes.c_int32)), ("stride", ctypes.POINTER(ctypes.c_int32)),
                ("weight", ctypes.c_void_p)]


class _PlanInfo(ctypes.Structure):
    _fields_ = [("variant", ctypes.c_int32), ("tile_rows", ctypes.c_int32), ("tile_cols", ctypes.c_int32),
                ("filters_per_warp", ctypes.c_int32), ("warps_per_cta", ctypes.c_int32),
                ("channels_per_stage", ctypes.c_int32), ("channel_splits", ctypes.c_int32),
                ("grid_x", ctypes.c_int32), ("grid_y", ctypes.c_int32), ("grid_z", ctypes.c_int32),
                ("smem_bytes", ctypes.c_int32), ("device_bytes", ctypes.c_int64), ("entries", ctypes.c_int64),
                ("generated", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_lib = None


def load() -> ctypes.CDLL:
    """Load ``libpatdnn.so`` (built in-tree by ``paper_2001_00138_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2001_00138_b200.build` "
                                "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.patdnn_encode.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_uint8),
                                  ctypes.POINTER(ctypes.c_uint16), i32, ctypes.POINTER(_Desc), ctypes.POINTER(vp)]
    lib.patdnn_conv.argtypes = [vp, vp, vp, vp]
    lib.patdnn_conv_host.argtypes = [vp, vp, vp, vp]
    lib.patdnn_conv_static.argtypes = [vp, vp, vp, vp]
    lib.patdnn_free.argtypes = [vp]
    lib.patdnn_check.argtypes = [vp]
    lib.patdnn_debug_wait.argtypes = [vp, ctypes.c_uint32, i32]
    lib.patdnn_export.argtypes = [vp, ctypes.POINTER(_FkwView)]
    lib.patdnn_decode.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.patdnn_plan.argtypes = [vp, ctypes.POINTER(_PlanInfo)]
    lib.patdnn_stack_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(i32), i32, ctypes.POINTER(vp)]
    lib.patdnn_stack_run.argtypes = [vp, vp, vp, vp]
    lib.patdnn_stack_run_host.argtypes = [vp, vp, vp, vp]
    lib.patdnn_stack_run_timed.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ctypes.c_float)]
    lib.patdnn_stack_submit_host.argtypes = [vp, vp, vp, vp]
    lib.patdnn_stack_wait_host.argtypes = [vp]
    lib.patdnn_stack_out_shape.argtypes = [vp] + [ctypes.POINTER(i32)] * 4
    lib.patdnn_stack_generated.argtypes = [vp, ctypes.POINTER(i32)]
    lib.patdnn_stack_free.argtypes = [vp]
    lib.patdnn_maxpool2x2.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp]
    lib.patdnn_launch_count.restype = ctypes.c_int64
    lib.patdnn_reset_launch_count.restype = None
    for name in ("patdnn_strerror", "patdnn_last_cuda_error", "patdnn_version"):
        getattr(lib, name).restype = ctypes.c_char_p
    lib.patdnn_strerror.argtypes = [i32]
    _lib = lib
    return lib


def _check(rc: int, where: str) -> None:
    if rc != OK:
        lib = load()
        detail = lib.patdnn_strerror(rc).decode()
        if rc == 6:
            detail += "; " + lib.patdnn_last_cuda_error().decode()
        raise PatdnnError(rc, where, detail)


def _ptr(x) -> int:
    """Raw address of a device buffer: an int, or anything with ``data_ptr()``."""
    return int(x.data_ptr()) if hasattr(x, "data_ptr") else int(x)


class Layer:
    """One encoded layer (``patdnn_handle``)."""

    def __init__(self, handle: int, desc: _Desc, keepalive):
        self._h = handle
        self.desc = desc
        self._keep = keepalive

    @property
    def handle(self) -> int:
        return self._h

    def conv(self, x, out, stream: int = 0) -> None:
        """patdnn_conv: x, out are device buffers (NCHW); asynchronous on ``stream`` (a cudaStream_t value)."""
        _check(load().patdnn_conv(self._h, _ptr(x), _ptr(out), stream), "patdnn_conv")

    def conv_static(self, x, out, stream: int = 0) -> None:
        """patdnn_conv_static: like :meth:`conv`, but the layer's scratch is the library's fixed 16 MiB device array,
        so the call allocates nothing (for callers that may not allocate device memory while running).  Calls that
        can overlap on the GPU must be serialised by the caller; make the first call before any stream capture."""
        _check(load().patdnn_conv_static(self._h, _ptr(x), _ptr(out), stream), "patdnn_conv_static")

    def conv_host(self, x: np.ndarray, out: np.ndarray, stream: int = 0) -> None:
        """patdnn_conv_host: host buffers in, host buffers out (copies inside the call)."""
        assert x.flags.c_contiguous and out.flags.c_contiguous
        _check(load().patdnn_conv_host(self._h, x.ctypes.data, out.ctypes.data, stream), "patdnn_conv_host")

    def check(self) -> None:
        """patdnn_check: synchronise and raise if a device-side bounded wait expired."""
        _check(load().patdnn_check(self._h), "patdnn_check")

    def debug_wait(self, polls: int, skip_load_iteration: int = 0) -> None:
        """patdnn_debug_wait: bound of the device-side waits (polls; 0 = default) and the test hook that withholds one
        iteration's loads so that a wait runs out."""
        _check(load().patdnn_debug_wait(self._h, polls, skip_load_iteration), "patdnn_debug_wait")

    def export(self) -> Dict[str, np.ndarray]:
        v = _FkwView()
        _check(load().patdnn_export(self._h, ctypes.byref(v)), "patdnn_export")
        F, P, K = v.F, v.P, v.K

        def arr(ptr, n, dt=np.int32):
            if n == 0:
                return np.zeros(0, dtype=dt)
            return np.ctypeslib.as_array(ptr, shape=(n,)).astype(dt, copy=True)

        if self.desc.dtype == F16:
            wt = np.ctypeslib.as_array(ctypes.cast(v.weight, ctypes.POINTER(ctypes.c_uint16)),
                                       shape=(max(K, 1) * 4,))[:K * 4].copy().reshape(K, 4)
        else:
            wt = np.ctypeslib.as_array(ctypes.cast(v.weight, ctypes.POINTER(ctypes.c_float)),
                                       shape=(max(K, 1) * 4,))[:K * 4].copy().reshape(K, 4)
        return {"offset": arr(v.offset, F + 1), "reorder": arr(v.reorder, F), "index": arr(v.index, K),
                "stride": arr(v.stride, F * (P + 1)).reshape(F, P + 1), "weight": wt}

    def decode(self) -> np.ndarray:
        out = np.empty((self.desc.F, self.desc.C, 3, 3), dtype=np.float32)
        _check(load().patdnn_decode(self._h, out.ctypes.data_as(ctypes.POINTER(ctypes.c_float))), "patdnn_decode")
        return out

    def plan(self) -> Dict[str, int]:
        info = _PlanInfo()
        _check(load().patdnn_plan(self._h, ctypes.byref(info)), "patdnn_plan")
        return {name: int(getattr(info, name)) for name, _ in _PlanInfo._fields_}

    def free(self) -> None:
        if self._h:
            load().patdnn_free(self._h)
            self._h = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def encode(weights: np.ndarray, mask: np.ndarray, pattern_set: Sequence[int], *, N: int, H: int, W: int,
           dtype: int = F32, relu: bool = True, bias: Optional[np.ndarray] = None,
           order: Optional[Sequence[int]] = None, variant: int = VARIANT_AUTO, host_only: bool = False) -> Layer:
    """patdnn_encode: validate, reorder (FKR), build FKW, plan and upload.  Returns a :class:`Layer`."""
    lib = load()
    w = np.ascontiguousarray(weights, dtype=np.float32)
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    pats = np.ascontiguousarray(pattern_set, dtype=np.uint16)
    if w.ndim != 4 or w.shape[2:] != (3, 3) or m.shape != w.shape:
        raise ValueError("weights and mask must both be [F, C, 3, 3]")
    F, C = w.shape[:2]
    desc = _Desc(F=F, C=C, N=N, H=H, W=W, dtype=dtype, relu=int(bool(relu)), variant=variant,
                 flags=FLAG_HOST_ONLY if host_only else 0)
    keep = [w, m, pats]
    if order is not None:
        o = np.ascontiguousarray(order, dtype=np.int32)
        if o.shape != (F,):
            raise ValueError("order must have F entries")
        desc.filter_order = 1
        desc.order = o.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
        keep.append(o)
    if bias is not None:
        b = np.ascontiguousarray(bias, dtype=np.float32)
        if b.shape != (F,):
            raise ValueError("bias must have F entries")
        desc.bias = b.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
        keep.append(b)
    h = ctypes.c_void_p()
    rc = lib.patdnn_encode(w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                           m.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                           pats.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), len(pats), ctypes.byref(desc),
                           ctypes.byref(h))
    _check(rc, "patdnn_encode")
    desc.order = None
    desc.bias = None
    return Layer(h.value, desc, None)


class Stack:
    """A chain of layers with optional 2x2 max-pools (``patdnn_stack``)."""

    def __init__(self, layers: Sequence[Layer], pool_after: Optional[Sequence[int]] = None):
        lib = load()
        n = len(layers)
        arr = (ctypes.c_void_p * n)(*[l.handle for l in layers])
        pools = (ctypes.c_int32 * n)(*([int(bool(p)) for p in pool_after] if pool_after is not None else [0] * n))
        h = ctypes.c_void_p()
        _check(lib.patdnn_stack_create(arr, pools, n, ctypes.byref(h)), "patdnn_stack_create")
        self._h = h.value
        self._layers = list(layers)        # the handles must outlive the stack

    def out_shape(self):
        v = [ctypes.c_int32() for _ in range(4)]
        _check(load().patdnn_stack_out_shape(self._h, *[ctypes.byref(x) for x in v]), "patdnn_stack_out_shape")
        return tuple(int(x.value) for x in v)

    def generated(self) -> int:
        """Number of layers of the stack that run code generated for them at stack creation."""
        v = ctypes.c_int32()
        _check(load().patdnn_stack_generated(self._h, ctypes.byref(v)), "patdnn_stack_generated")
        return int(v.value)

    def run(self, x, out, stream: int = 0) -> None:
        _check(load().patdnn_stack_run(self._h, _ptr(x), _ptr(out), stream), "patdnn_stack_run")

    def run_timed(self, x, out, stream: int = 0) -> np.ndarray:
        """patdnn_stack_run_timed: one synchronous pass; returns the milliseconds each layer took inside the stack."""
        ms = np.zeros(len(self._layers), dtype=np.float32)
        _check(load().patdnn_stack_run_timed(self._h, _ptr(x), _ptr(out), stream,
                                             ms.ctypes.data_as(ctypes.POINTER(ctypes.c_float))), "patdnn_stack_run_timed")
        return ms

    def run_host(self, x: np.ndarray, out: np.ndarray, stream: int = 0) -> None:
        assert x.flags.c_contiguous and out.flags.c_contiguous
        _check(load().patdnn_stack_run_host(self._h, x.ctypes.data, out.ctypes.data, stream), "patdnn_stack_run_host")

    def submit_host(self, x: np.ndarray, out: np.ndarray, stream: int = 0) -> None:
        """Pipelined run_host: returns at once; at most two batches in flight; pair every call with wait_host()."""
        assert x.flags.c_contiguous and out.flags.c_contiguous
        _check(load().patdnn_stack_submit_host(self._h, x.ctypes.data, out.ctypes.data, stream), "patdnn_stack_submit_host")

    def wait_host(self) -> None:
        _check(load().patdnn_stack_wait_host(self._h), "patdnn_stack_wait_host")

    def free(self) -> None:
        if self._h:
            load().patdnn_stack_free(self._h)
            self._h = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def maxpool2x2(x, out, N: int, C: int, H: int, W: int, dtype: int = F32, stream: int = 0) -> None:
    _check(load().patdnn_maxpool2x2(_ptr(x), _ptr(out), N, C, H, W, dtype, stream), "patdnn_maxpool2x2")


def launch_count() -> int:
    return int(load().patdnn_launch_count())


def reset_launch_count() -> None:
    load().patdnn_reset_launch_count()


def version() -> str:
    return load().patdnn_version().decode()
