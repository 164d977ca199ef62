"""CPU oracle for the forward grouped convolution.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product path (the CUDA library and its Python binding) never does, and nothing here imports the
product path.  The arithmetic lives in ``gconv_ref.c`` (seven loops, fp64 accumulation; grouped
convolution of Section II and the convolution stage of Algorithm 1 of the paper); this module only
compiles that file with gcc and marshals numpy arrays to it.

``gspc.c`` is a second, separate CPU program: the paper's own method (Algorithm 1, Section III-B: kernel reshaping,
input reshaping, convolution on the packed volumes, output reshaping, with tile sizes T_I and T_O) in float32.  It is
not the oracle -- the tests pin it against ``gconv_ref`` -- it is the CPU baseline the benchmark times beside it.
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


_GSPC_SRC = os.path.join(_HERE, "gspc.c")
_GSPC_LIB = os.path.join(_HERE, "libgspc.so")
_gspc = None


def _compile(src: str, lib: str, opt: str, force: bool) -> str:
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(src):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", opt, "-fopenmp", "-shared", "-fPIC", "-o", tmp, src])
    os.replace(tmp, lib)
    return lib


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2, OpenMP) and the GSPC baseline (gcc -O3, OpenMP) into shared objects beside
    their sources; returns the oracle's path."""
    _compile(_GSPC_SRC, _GSPC_LIB, "-O3", force)
    return _compile(_SRC, _LIB, "-O2", force)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.gconv_ref_f64.restype = ctypes.c_int
            lib.gconv_ref_f64.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 11 + [
                ctypes.c_int, ctypes.POINTER(ctypes.c_longlong)]
            lib.gconv_ref_f64_2d.restype = ctypes.c_int
            lib.gconv_ref_f64_2d.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 14 + [
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


def _pair(v):
    """An int stands for both axes; a pair is (rows, columns)."""
    if isinstance(v, (tuple, list)):
        if len(v) != 2:
            raise ValueError("a per-axis parameter is (rows, columns)")
        return int(v[0]), int(v[1])
    return int(v), int(v)


def gconv_ref(x: np.ndarray, w: np.ndarray, stride=1, pad=0, dilation=1,
              groups: int = 1, threads: int = 1, return_macs: bool = False):
    """Grouped convolution y = gconv(x, w) in fp64.

    x: float32 [N, C_in, H, W]; w: float32 [C_out, C_in/groups, KH, KW]; returns float64
    [N, C_out, H_out, W_out] (and the MAC count of Eq. (2) when ``return_macs``).  stride, pad and dilation are
    ints (both axes) or (rows, columns) pairs, as Algorithm 1's S_h and S_w.
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
    (sh, sw), (ph, pw), (dh, dw) = _pair(stride), _pair(pad), _pair(dilation)
    Ho = out_dim(H, KH, sh, ph, dh)
    Wo = out_dim(W, KW, sw, pw, dw)
    if Ho < 1 or Wo < 1:
        raise ValueError("empty output")
    y = np.empty((N, C_out, Ho, Wo), dtype=np.float64)
    macs = ctypes.c_longlong(0)
    if (sh, ph, dh) == (sw, pw, dw):
        rc = lib.gconv_ref_f64(x.ctypes.data, w.ctypes.data, y.ctypes.data, N, C_in, H, W, C_out, KH, KW,
                               sh, ph, dh, groups, int(threads), ctypes.byref(macs))
    else:
        rc = lib.gconv_ref_f64_2d(x.ctypes.data, w.ctypes.data, y.ctypes.data, N, C_in, H, W, C_out, KH, KW,
                                  sh, sw, ph, pw, dh, dw, groups, int(threads), ctypes.byref(macs))
    if rc != 0:
        raise ValueError("gconv_ref_f64 rejected the problem")
    return (y, int(macs.value)) if return_macs else y


def _load_gspc():
    global _gspc
    with _lock:
        if _gspc is None:
            build()
            lib = ctypes.CDLL(_GSPC_LIB)
            lib.gspc_packed_kernel_elems.restype = ctypes.c_size_t
            lib.gspc_packed_kernel_elems.argtypes = [ctypes.c_int] * 5
            lib.gspc_pack_kernels.restype = ctypes.c_int
            lib.gspc_pack_kernels.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 7
            lib.gspc_forward_f32.restype = ctypes.c_int
            lib.gspc_forward_f32.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 14 + [
                ctypes.POINTER(ctypes.c_double)]
            _gspc = lib
    return _gspc


def gspc_pack_kernels(w: np.ndarray, groups: int, T_I: int, T_O: int) -> np.ndarray:
    """Stage 1 of Algorithm 1 (kernel reshaping; done ahead of time): w [C_out, CPG, KH, KW] -> the 7-D volume
    [g, KPG/T_O, CPG/T_I, KH, KW, T_I, T_O], returned flat."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    C_out, Cg, KH, KW = w.shape
    wp = np.empty(w.size, dtype=np.float32)
    rc = _load_gspc().gspc_pack_kernels(w.ctypes.data, wp.ctypes.data, Cg * groups, C_out, KH, KW, groups, T_I, T_O)
    if rc != 0:
        raise ValueError("tile sizes must divide CPG and KPG (Eq. (1) bounds them by CPG and KPG)")
    return wp


def gspc_forward(x: np.ndarray, wp: np.ndarray, w_shape, stride: int, pad: int, dilation: int, groups: int, T_I: int, T_O: int,
                 threads: int = 1, return_stage_seconds: bool = False):
    """Stages 2-4 of Algorithm 1 in float32 on kernels packed by gspc_pack_kernels with the same tiles."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    N, C_in, H, W = x.shape
    C_out, Cg, KH, KW = w_shape
    Ho = out_dim(H, KH, stride, pad, dilation)
    Wo = out_dim(W, KW, stride, pad, dilation)
    y = np.empty((N, C_out, Ho, Wo), dtype=np.float32)
    secs = (ctypes.c_double * 3)()
    rc = _load_gspc().gspc_forward_f32(x.ctypes.data, wp.ctypes.data, y.ctypes.data, N, C_in, H, W, C_out, KH, KW, stride, pad,
                                       dilation, groups, T_I, T_O, int(threads), secs)
    if rc != 0:
        raise ValueError("gspc_forward_f32 rejected the problem (%d)" % rc)
    return (y, tuple(secs)) if return_stage_seconds else y
