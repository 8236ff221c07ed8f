"""ctypes binding of libsinglequant.so: the same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's kernels; PyTorch appears here only as the owner
of device memory and streams.  Loading fails loudly when the shared library is missing: there
is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (POINTER, byref, c_char_p, c_double, c_float, c_int32, c_int64, c_size_t,
                    c_uint32, c_uint64, c_void_p)
from typing import Optional, Tuple

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsinglequant.so")

SQ_OK = 0
SQ_ERR_INVALID_ARG, SQ_ERR_SHAPE, SQ_ERR_ALIGN, SQ_ERR_UNSUPPORTED = 1, 2, 3, 4
SQ_ERR_NOMEM, SQ_ERR_CUDA, SQ_ERR_TIMEOUT = 5, 6, 7
SQ_ROT_ART, SQ_ROT_URT, SQ_ROT_HADAMARD, SQ_ROT_DEFAULT = 1, 2, 4, 7
SQ_ROT_APPLY_STRUCTURED = 1 << 20
SQ_ROT_FUSE_DECODE = 1 << 21

EXPORTS = (
    "sq_factorize", "sq_build_rotation", "sq_rotation_from_factors", "sq_rotation_get_factors",
    "sq_rotation_dims", "sq_rotation_is_structured", "sq_rotation_destroy", "sq_rotate_quant_act", "sq_pack_weight",
    "sq_w4a4_gemm", "sq_linear_workspace_bytes", "sq_linear",
    "sq_linear_static", "sq_linear_host_workspace_bytes", "sq_linear_host", "sq_last_device_status",
    "sq_debug_bounded_wait", "sq_kernel_launch_count", "sq_status_string",
    "sq_pack_weight_wo", "sq_rotate_act_f16", "sq_w4a16_gemm", "sq_linear_wo_workspace_bytes", "sq_linear_wo",
    "sq_linear_grouped",
)


class SingleQuantError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """Loads the C-ABI library (built by `python -m paper_2511_22316_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_22316_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.sq_factorize.argtypes = [c_int64, POINTER(c_int32), POINTER(c_int32)]
    lib.sq_build_rotation.argtypes = [c_void_p, c_int64, c_int64, c_int32, c_int32, c_uint32, c_uint64,
                                      c_void_p, POINTER(c_void_p)]
    lib.sq_rotation_from_factors.argtypes = [c_void_p, c_void_p, c_int32, c_int32, POINTER(c_void_p)]
    lib.sq_rotation_get_factors.argtypes = [c_void_p, c_void_p, c_void_p]
    lib.sq_rotation_dims.argtypes = [c_void_p, POINTER(c_int32), POINTER(c_int32)]
    lib.sq_rotation_is_structured.argtypes = [c_void_p]
    lib.sq_rotation_is_structured.restype = c_int32
    lib.sq_rotation_destroy.argtypes = [c_void_p]
    lib.sq_rotation_destroy.restype = None
    lib.sq_rotate_quant_act.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.sq_pack_weight.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p]
    lib.sq_w4a4_gemm.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64,
                                 c_void_p, c_void_p, c_void_p]
    lib.sq_linear_workspace_bytes.argtypes = [c_int64, c_int64]
    lib.sq_linear_workspace_bytes.restype = c_size_t
    lib.sq_linear.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_int64, c_int64,
                              c_void_p, c_size_t, c_void_p, c_void_p]
    lib.sq_linear_static.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_int64, c_int64,
                                     c_void_p, c_void_p]
    lib.sq_linear_host_workspace_bytes.argtypes = [c_int64, c_int64, c_int64]
    lib.sq_linear_host_workspace_bytes.restype = c_size_t
    lib.sq_linear_host.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_int64, c_int64,
                                   c_void_p, c_size_t, c_void_p, c_void_p]
    lib.sq_pack_weight_wo.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int32, c_void_p, c_void_p, c_void_p]
    lib.sq_rotate_act_f16.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p]
    lib.sq_w4a16_gemm.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p]
    lib.sq_linear_wo_workspace_bytes.argtypes = [c_int64, c_int64]
    lib.sq_linear_wo_workspace_bytes.restype = c_size_t
    lib.sq_linear_wo.argtypes = [c_void_p, c_void_p, c_int64, c_void_p, c_void_p, c_int64, c_int64,
                                 c_void_p, c_size_t, c_void_p, c_void_p]
    lib.sq_linear_grouped.argtypes = [POINTER(c_void_p), c_int32, POINTER(c_int64), c_void_p, POINTER(c_void_p),
                                      POINTER(c_void_p), c_int64, c_int64, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.sq_last_device_status.argtypes = [c_void_p]
    lib.sq_debug_bounded_wait.argtypes = [c_uint32, c_void_p]
    lib.sq_kernel_launch_count.argtypes = []
    lib.sq_kernel_launch_count.restype = c_uint64
    lib.sq_status_string.argtypes = [ctypes.c_int]
    lib.sq_status_string.restype = c_char_p
    for name in EXPORTS:
        getattr(lib, name)          # raises AttributeError if the library lacks an entry point
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().sq_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != SQ_OK:
        raise SingleQuantError(code, where)


def _ptr(t) -> Optional[int]:
    """Device (torch tensor) or host (numpy array) pointer; None stays NULL."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    if isinstance(t, int):
        return t
    return t.data_ptr()


_torch = None


def _stream(stream) -> Optional[int]:
    if stream is None:
        global _torch
        if _torch is None:
            import torch
            _torch = torch
        return _torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


class Rotation:
    """Owns a sq_rotation_t handle."""

    def __init__(self, handle: int):
        self._h = c_void_p(handle)

    @property
    def handle(self) -> c_void_p:
        return self._h

    @property
    def dims(self) -> Tuple[int, int]:
        a, b = c_int32(), c_int32()
        _check(load().sq_rotation_dims(self._h, byref(a), byref(b)), "sq_rotation_dims")
        return a.value, b.value

    def factors(self) -> Tuple[np.ndarray, np.ndarray]:
        return sq_rotation_get_factors(self)

    @property
    def structured(self) -> bool:
        return sq_rotation_is_structured(self)

    def close(self) -> None:
        if self._h:
            load().sq_rotation_destroy(self._h)
            self._h = c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def sq_factorize(n: int) -> Tuple[int, int]:
    a, b = c_int32(), c_int32()
    _check(load().sq_factorize(int(n), byref(a), byref(b)), "sq_factorize")
    return a.value, b.value


def SQ_ROT_ART_STEPS(k: int) -> int:
    """Flag bits for k >= 1 ART steps (OR into `flags`)."""
    return (int(k) - 1) << 8


def sq_build_rotation(calib: np.ndarray, n1: int, n2: int, flags: int = SQ_ROT_DEFAULT, seed: int = 0,
                      O: Optional[np.ndarray] = None) -> Rotation:
    calib = np.ascontiguousarray(calib, dtype=np.float32)
    T, n = calib.shape
    if O is not None:
        O = np.ascontiguousarray(O, dtype=np.float64)
    out = c_void_p()
    _check(load().sq_build_rotation(calib.ctypes.data, T, n, n1, n2, flags, seed,
                                    None if O is None else O.ctypes.data, byref(out)), "sq_build_rotation")
    return Rotation(out.value)


def sq_rotation_from_factors(R1: np.ndarray, R2: np.ndarray) -> Rotation:
    R1 = np.ascontiguousarray(R1, dtype=np.float32)
    R2 = np.ascontiguousarray(R2, dtype=np.float32)
    out = c_void_p()
    _check(load().sq_rotation_from_factors(R1.ctypes.data, R2.ctypes.data, R1.shape[0], R2.shape[0], byref(out)),
           "sq_rotation_from_factors")
    return Rotation(out.value)


def sq_rotation_get_factors(rot: Rotation) -> Tuple[np.ndarray, np.ndarray]:
    n1, n2 = rot.dims
    R1 = np.empty((n1, n1), np.float32)
    R2 = np.empty((n2, n2), np.float32)
    _check(load().sq_rotation_get_factors(rot.handle, R1.ctypes.data, R2.ctypes.data), "sq_rotation_get_factors")
    return R1, R2


def sq_rotation_is_structured(rot: Rotation) -> bool:
    return bool(load().sq_rotation_is_structured(rot.handle))


def sq_rotate_quant_act(rot: Rotation, X, M: int, Xq, sx, Zdbg=None, stream=None) -> None:
    _check(load().sq_rotate_quant_act(rot.handle, _ptr(X), M, _ptr(Xq), _ptr(sx), _ptr(Zdbg), _stream(stream)),
           "sq_rotate_quant_act")


def sq_pack_weight(rot: Optional[Rotation], W, N: int, K: int, Wq, sw, stream=None) -> None:
    _check(load().sq_pack_weight(None if rot is None else rot.handle, _ptr(W), N, K, _ptr(Wq), _ptr(sw),
                                 _stream(stream)), "sq_pack_weight")


def sq_w4a4_gemm(Xq, sx, Wq, sw, M: int, N: int, K: int, Y, accdbg=None, stream=None) -> None:
    _check(load().sq_w4a4_gemm(_ptr(Xq), _ptr(sx), _ptr(Wq), _ptr(sw), M, N, K, _ptr(Y), _ptr(accdbg),
                               _stream(stream)), "sq_w4a4_gemm")


def sq_linear_workspace_bytes(M: int, K: int) -> int:
    return int(load().sq_linear_workspace_bytes(M, K))


def sq_linear(rot: Rotation, X, M: int, Wq, sw, N: int, K: int, workspace, workspace_bytes: int, Y,
              stream=None) -> None:
    _check(load().sq_linear(rot.handle, _ptr(X), M, _ptr(Wq), _ptr(sw), N, K, _ptr(workspace), workspace_bytes,
                            _ptr(Y), _stream(stream)), "sq_linear")


SQ_LINEAR_STATIC_SCRATCH_BYTES = 8 << 20


def sq_linear_static(rot: Rotation, X, M: int, Wq, sw, N: int, K: int, Y, stream=None) -> None:
    """sq_linear with the library's built-in scratch: no workspace argument, no allocation on the
    call path (for callers that cannot allocate device memory; see the header).  Problems whose
    workspace exceeds SQ_LINEAR_STATIC_SCRATCH_BYTES raise SingleQuantError(SQ_ERR_UNSUPPORTED)."""
    _check(load().sq_linear_static(rot.handle, _ptr(X), M, _ptr(Wq), _ptr(sw), N, K, _ptr(Y), _stream(stream)),
           "sq_linear_static")


def sq_linear_host_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(load().sq_linear_host_workspace_bytes(M, N, K))


def sq_linear_host(rot: Rotation, X_host, M: int, Wq, sw, N: int, K: int, workspace, workspace_bytes: int,
                   Y_host, stream=None) -> None:
    _check(load().sq_linear_host(rot.handle, _ptr(X_host), M, _ptr(Wq), _ptr(sw), N, K, _ptr(workspace),
                                 workspace_bytes, _ptr(Y_host), _stream(stream)), "sq_linear_host")


def sq_pack_weight_wo(rot: Optional[Rotation], W, N: int, K: int, bits: int, Wq, sw, stream=None) -> None:
    """Offline weight path of the weight-only variant: `bits` = 4 or 3, codes in the weight-only order."""
    _check(load().sq_pack_weight_wo(None if rot is None else rot.handle, _ptr(W), N, K, int(bits), _ptr(Wq),
                                    _ptr(sw), _stream(stream)), "sq_pack_weight_wo")


def sq_rotate_act_f16(rot: Rotation, X, M: int, Z16, stream=None) -> None:
    _check(load().sq_rotate_act_f16(rot.handle, _ptr(X), M, _ptr(Z16), _stream(stream)), "sq_rotate_act_f16")


def sq_w4a16_gemm(Z16, Wq, sw, M: int, N: int, K: int, Y, stream=None) -> None:
    _check(load().sq_w4a16_gemm(_ptr(Z16), _ptr(Wq), _ptr(sw), M, N, K, _ptr(Y), _stream(stream)), "sq_w4a16_gemm")


def sq_linear_wo_workspace_bytes(M: int, K: int) -> int:
    return int(load().sq_linear_wo_workspace_bytes(M, K))


def sq_linear_wo(rot: Rotation, X, M: int, Wq, sw, N: int, K: int, workspace, workspace_bytes: int, Y,
                 stream=None) -> None:
    _check(load().sq_linear_wo(rot.handle, _ptr(X), M, _ptr(Wq), _ptr(sw), N, K, _ptr(workspace), workspace_bytes,
                               _ptr(Y), _stream(stream)), "sq_linear_wo")


def sq_linear_grouped(rots, offsets, X, Wq, sw, N: int, K: int, workspace, workspace_bytes: int, Y,
                      stream=None) -> None:
    """The W4A4 layer of a mixture-of-experts block: `rots`, `Wq`, `sw` are sequences with one entry per
    expert, `offsets` the E + 1 row offsets of the expert-sorted tokens."""
    E = len(rots)
    h = (c_void_p * E)(*[r.handle for r in rots])
    off = (c_int64 * (E + 1))(*[int(o) for o in offsets])
    wq = (c_void_p * E)(*[_ptr(w) for w in Wq])
    sws = (c_void_p * E)(*[_ptr(w) for w in sw])
    _check(load().sq_linear_grouped(h, E, off, _ptr(X), wq, sws, N, K, _ptr(workspace), workspace_bytes, _ptr(Y),
                                    _stream(stream)), "sq_linear_grouped")


def sq_last_device_status(stream=None) -> int:
    return int(load().sq_last_device_status(_stream(stream)))


def sq_debug_bounded_wait(polls: int, stream=None) -> None:
    """Enqueues the diagnostic kernel whose only wait runs out after `polls` polls (see the header)."""
    _check(load().sq_debug_bounded_wait(int(polls), _stream(stream)), "sq_debug_bounded_wait")


def sq_kernel_launch_count() -> int:
    return int(load().sq_kernel_launch_count())
