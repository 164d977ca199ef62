"""ctypes binding of the libgconv C ABI (include/gconv.h): same names, argument marshalling only.

Every step of the convolution runs inside the CUDA library.  There is no fallback: if the shared
library has not been built, importing a function from here raises.  torch is used by callers for
device memory and streams; this module accepts raw integer pointers or anything with
``data_ptr()`` / ``cuda_stream``.
"""
from __future__ import annotations

import ctypes
import os

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgconv.so")
_lib = None

GCONV_OK = 0
GCONV_ERR_NULL = 1
GCONV_ERR_INVALID_ARG = 2
GCONV_ERR_UNSUPPORTED = 3
GCONV_ERR_ALIGNMENT = 4
GCONV_ERR_CUDA = 5
GCONV_ERR_PACK_MISMATCH = 6
GCONV_ERR_TIMEOUT = 7
GCONV_ERR_TOO_LARGE = 8
GCONV_ERR_WORKSPACE = 9

GCONV_VARIANT_AUTO = 0
GCONV_VARIANT_DIRECT_GENERIC = 1
GCONV_VARIANT_DIRECT_TILED = 2
GCONV_VARIANT_IGEMM_TF32 = 3

# tolerance on max|y - y_ref| / max|y_ref| that goes with each variant
VARIANT_TOLERANCE = {GCONV_VARIANT_DIRECT_GENERIC: 1e-5, GCONV_VARIANT_DIRECT_TILED: 1e-5,
                     GCONV_VARIANT_IGEMM_TF32: 5e-3}

_vp = ctypes.c_void_p
_SIGNATURES = {
    "gconv_desc_create": (ctypes.c_int, [ctypes.POINTER(_vp)] + [ctypes.c_int] * 11),
    "gconv_desc_create_2d": (ctypes.c_int, [ctypes.POINTER(_vp)] + [ctypes.c_int] * 14),
    "gconv_desc_destroy": (ctypes.c_int, [_vp]),
    "gconv_out_shape": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]),
    "gconv_macs": (ctypes.c_longlong, [_vp]),
    "gconv_packed_bytes": (ctypes.c_size_t, [_vp]),
    "gconv_variant": (ctypes.c_int, [_vp]),
    "gconv_variant_supported": (ctypes.c_int, [_vp, ctypes.c_int]),
    "gconv_desc_set_variant": (ctypes.c_int, [_vp, ctypes.c_int]),
    "gconv_pack_weights": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "gconv_forward": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "gconv_forward_host": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "gconv_forward_host_static": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp]),
    "gconv_block_supported": (ctypes.c_int, [_vp, ctypes.c_int]),
    "gconv_block_packed_bytes": (ctypes.c_size_t, [_vp, ctypes.c_int]),
    "gconv_block_pack_weights": (ctypes.c_int, [_vp, ctypes.c_int, _vp, _vp, _vp, _vp]),
    "gconv_block_forward": (ctypes.c_int, [_vp, ctypes.c_int, _vp, _vp, _vp, _vp]),
    "gconv_forward_launches": (ctypes.c_int, [_vp]),
    "gconv_workspace_bytes": (ctypes.c_size_t, [_vp]),
    "gconv_desc_set_workspace": (ctypes.c_int, [_vp, _vp, ctypes.c_size_t]),
    "gconv_desc_set_debug": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int]),
    "gconv_last_status": (ctypes.c_int, [_vp, _vp]),
    "gconv_last_cuda_error": (ctypes.c_int, [_vp]),
    "gconv_last_status_detail": (ctypes.c_int, [_vp]),
    "gconv_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "gconv_variant_name": (ctypes.c_char_p, [ctypes.c_int]),
}


class GconvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


def lib_path() -> str:
    return _LIB_PATH


def load() -> ctypes.CDLL:
    """Load libgconv.so (built in-tree by ``paper_2006_09791_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("libgconv.so is not built: run `python -m paper_2006_09791_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


def _stream(s) -> int:
    if s is None:
        return 0
    if isinstance(s, int):
        return s
    return int(s.cuda_stream)


def _check(rc: int, where: str) -> None:
    if rc != GCONV_OK:
        raise GconvError(rc, where)


def status_string(status: int) -> str:
    return load().gconv_status_string(int(status)).decode()


def variant_name(variant: int) -> str:
    return load().gconv_variant_name(int(variant)).decode()


def gconv_desc_create(N, C_in, H, W, C_out, KH, KW, stride, pad, dilation, groups) -> int:
    h = _vp(0)
    rc = load().gconv_desc_create(ctypes.byref(h), N, C_in, H, W, C_out, KH, KW, stride, pad, dilation, groups)
    _check(rc, "gconv_desc_create")
    return h.value


def gconv_desc_create_2d(N, C_in, H, W, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w, dilation_h, dilation_w, groups) -> int:
    h = _vp(0)
    rc = load().gconv_desc_create_2d(ctypes.byref(h), N, C_in, H, W, C_out, KH, KW, stride_h, stride_w, pad_h, pad_w,
                                     dilation_h, dilation_w, groups)
    _check(rc, "gconv_desc_create_2d")
    return h.value


def gconv_desc_destroy(desc) -> None:
    _check(load().gconv_desc_destroy(desc), "gconv_desc_destroy")


def gconv_out_shape(desc):
    ho, wo = ctypes.c_int(0), ctypes.c_int(0)
    _check(load().gconv_out_shape(desc, ctypes.byref(ho), ctypes.byref(wo)), "gconv_out_shape")
    return ho.value, wo.value


def gconv_macs(desc) -> int:
    return int(load().gconv_macs(desc))


def gconv_packed_bytes(desc) -> int:
    return int(load().gconv_packed_bytes(desc))


def gconv_variant(desc) -> int:
    return int(load().gconv_variant(desc))


def gconv_variant_supported(desc, variant) -> bool:
    return bool(load().gconv_variant_supported(desc, int(variant)))


def gconv_desc_set_variant(desc, variant) -> None:
    _check(load().gconv_desc_set_variant(desc, int(variant)), "gconv_desc_set_variant")


def gconv_pack_weights(desc, w_ochw, w_packed, stream=None) -> None:
    _check(load().gconv_pack_weights(desc, _ptr(w_ochw), _ptr(w_packed), _stream(stream)), "gconv_pack_weights")


def gconv_forward(desc, x_nchw, w_packed, y_nchw, stream=None) -> None:
    _check(load().gconv_forward(desc, _ptr(x_nchw), _ptr(w_packed), _ptr(y_nchw), _stream(stream)), "gconv_forward")


def gconv_forward_host(desc, x_host, w_packed, y_host, x_stage, y_stage, stream=None) -> None:
    _check(load().gconv_forward_host(desc, _ptr(x_host), _ptr(w_packed), _ptr(y_host), _ptr(x_stage), _ptr(y_stage),
                                     _stream(stream)), "gconv_forward_host")


def gconv_forward_host_static(desc, x_host, w_packed, y_host, stream=None) -> None:
    """Host-buffer forward that allocates nothing (static device scratch, at most 16 MiB of x + y + workspace);
    blocks until y_host is complete and raises on any status other than GCONV_OK."""
    _check(load().gconv_forward_host_static(desc, _ptr(x_host), _ptr(w_packed), _ptr(y_host), _stream(stream)),
           "gconv_forward_host_static")


def gconv_block_supported(desc, C2: int) -> bool:
    return bool(load().gconv_block_supported(desc, int(C2)))


def gconv_block_packed_bytes(desc, C2: int) -> int:
    return int(load().gconv_block_packed_bytes(desc, int(C2)))


def gconv_block_pack_weights(desc, C2: int, w_ochw, w2, w_packed, stream=None) -> None:
    """Packs the grouped 3x3 weights and the pointwise weights [C2, C_out] of the fused block (asynchronous)."""
    _check(load().gconv_block_pack_weights(desc, int(C2), _ptr(w_ochw), _ptr(w2), _ptr(w_packed), _stream(stream)),
           "gconv_block_pack_weights")


def gconv_block_forward(desc, C2: int, x_nchw, w_packed, y2_nchw, stream=None) -> None:
    """Grouped 3x3 convolution followed by the pointwise convolution, one kernel (asynchronous)."""
    _check(load().gconv_block_forward(desc, int(C2), _ptr(x_nchw), _ptr(w_packed), _ptr(y2_nchw), _stream(stream)),
           "gconv_block_forward")


def gconv_forward_launches(desc) -> int:
    return int(load().gconv_forward_launches(desc))


def gconv_workspace_bytes(desc) -> int:
    return int(load().gconv_workspace_bytes(desc))


def gconv_desc_set_workspace(desc, workspace, nbytes: int) -> None:
    """Attach a caller-owned device workspace of `nbytes` bytes (None detaches)."""
    _check(load().gconv_desc_set_workspace(desc, _ptr(workspace), int(nbytes)), "gconv_desc_set_workspace")


def gconv_desc_set_debug(desc, wait_limit_us: int = 0, skip_stage: int = -1) -> None:
    _check(load().gconv_desc_set_debug(desc, int(wait_limit_us), int(skip_stage)), "gconv_desc_set_debug")


def gconv_last_status(desc, stream=None) -> int:
    return int(load().gconv_last_status(desc, _stream(stream)))


def gconv_last_cuda_error(desc) -> int:
    return int(load().gconv_last_cuda_error(desc))


def gconv_last_status_detail(desc) -> int:
    return int(load().gconv_last_status_detail(desc))
