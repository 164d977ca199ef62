"""CPU oracle for the forward grouped convolution.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product path (the CUDA library and its Python binding) never does, and nothing here imports the
product path.  The arithmetic lives in ``gconv_ref.c`` (seven loops, fp64 accumulation; grouped
convolution of Section II and the convolution stage of Algorithm 1 of the paper); this module only
compiles that file with gcc and marshals numpy arrays to it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gconv_ref.c")
_LIB = os.path.join(_HERE, "libgconv_ref.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object beside its source (gcc, -O2, OpenMP)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.gconv_ref_f64.restype = ctypes.c_int
            lib.gconv_ref_f64.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 11 + [
                ctypes.c_int, ctypes.POINTER(ctypes.c_longlong)]
            lib.gconv_ref_out_dim.restype = ctypes.c_int
            lib.gconv_ref_out_dim.argtypes = [ctypes.c_int] * 5
            lib.gconv_ref_max_threads.restype = ctypes.c_int
            _lib = lib
    return _lib


def out_dim(size: int, k: int, stride: int, pad: int, dilation: int = 1) -> int:
    """floor((size + 2*pad - dilation*(k-1) - 1)/stride) + 1, or 0 when the window does not fit."""
    return int(_load().gconv_ref_out_dim(size, k, stride, pad, dilation))


def max_threads() -> int:
    return int(_load().gconv_ref_max_threads())


def gconv_ref(x: np.ndarray, w: np.ndarray, stride: int = 1, pad: int = 0, dilation: int = 1,
              groups: int = 1, threads: int = 1, return_macs: bool = False):
    """Grouped convolution y = gconv(x, w) in fp64.

    x: float32 [N, C_in, H, W]; w: float32 [C_out, C_in/groups, KH, KW]; returns float64
    [N, C_out, H_out, W_out] (and the MAC count of Eq. (2) when ``return_macs``).
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    if x.ndim != 4 or w.ndim != 4:
        raise ValueError("x must be [N,C_in,H,W] and w [C_out,Cg,KH,KW]")
    N, C_in, H, W = x.shape
    C_out, Cg, KH, KW = w.shape
    if groups < 1 or C_in % groups or C_out % groups or C_in // groups != Cg:
        raise ValueError("channels must split evenly over groups and w.shape[1] == C_in/groups")
    lib = _load()
    Ho = out_dim(H, KH, stride, pad, dilation)
    Wo = out_dim(W, KW, stride, pad, dilation)
    if Ho < 1 or Wo < 1:
        raise ValueError("empty output")
    y = np.empty((N, C_out, Ho, Wo), dtype=np.float64)
    macs = ctypes.c_longlong(0)
    rc = lib.gconv_ref_f64(x.ctypes.data, w.ctypes.data, y.ctypes.data, N, C_in, H, W, C_out, KH, KW,
                           stride, pad, dilation, groups, int(threads), ctypes.byref(macs))
    if rc != 0:
        raise ValueError("gconv_ref_f64 rejected the problem")
    return (y, int(macs.value)) if return_macs else y
