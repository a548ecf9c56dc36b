"""ctypes loader for the C oracle (``conv_oracle.c``).  Test infrastructure only."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_conv.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (plain -O2, OpenMP over (image, filter); no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f32p = ctypes.POINTER(ctypes.c_float)
        u8p = ctypes.POINTER(ctypes.c_ubyte)
        lib.oracle_conv3x3.argtypes = [f32p, f32p, u8p, f32p] + [ctypes.c_int] * 6 + [f32p]
        lib.oracle_conv3x3.restype = ctypes.c_int
        lib.oracle_conv3x3_point.argtypes = [f32p, f32p, u8p, f32p] + [ctypes.c_int] * 8
        lib.oracle_conv3x3_point.restype = ctypes.c_double
        lib.oracle_maxpool2x2.argtypes = [f32p] + [ctypes.c_int] * 4 + [f32p]
        lib.oracle_maxpool2x2.restype = ctypes.c_int
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _u8(a):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_ubyte))


def conv3x3(x: np.ndarray, weights: np.ndarray, mask: np.ndarray, bias: Optional[np.ndarray], relu: bool) -> np.ndarray:
    """out[n,f,y,x] = act(bias[f] + sum_{c,r,s} (weights*mask)[f,c,r,s] * x[n,c,y+r-1,x+s-1]), zero padding."""
    N, C, H, W = x.shape
    F = weights.shape[0]
    assert weights.shape == (F, C, 3, 3) and mask.shape == (F, C, 3, 3)
    xa, xp = _f32(x)
    wa, wp = _f32(weights)
    ma, mp = _u8(mask)
    out = np.empty((N, F, H, W), dtype=np.float32)
    if bias is None:
        bp = ctypes.POINTER(ctypes.c_float)()
    else:
        ba, bp = _f32(bias)
        assert ba.shape == (F,)
    rc = _load().oracle_conv3x3(xp, wp, mp, bp, N, C, H, W, F, int(bool(relu)),
                                out.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    if rc != 0:
        raise RuntimeError(f"oracle_conv3x3 failed with status {rc}")
    return out


def conv3x3_point(x, weights, mask, bias, relu, n, f, y, xx) -> float:
    """A single output element by the same definition (double, unrounded)."""
    N, C, H, W = x.shape
    xa, xp = _f32(x)
    wa, wp = _f32(weights)
    ma, mp = _u8(mask)
    if bias is None:
        bp = ctypes.POINTER(ctypes.c_float)()
    else:
        ba, bp = _f32(bias)
    return float(_load().oracle_conv3x3_point(xp, wp, mp, bp, C, H, W, int(bool(relu)), n, f, y, xx))


def maxpool2x2(x: np.ndarray) -> np.ndarray:
    N, C, H, W = x.shape
    xa, xp = _f32(x)
    out = np.empty((N, C, H // 2, W // 2), dtype=np.float32)
    rc = _load().oracle_maxpool2x2(xp, N, C, H, W, out.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
    if rc != 0:
        raise RuntimeError("oracle_maxpool2x2 failed")
    return out


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))
