"""Thin ctypes binding of ``libhccs.so``: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/hccs.h``
and raises :class:`HccsError` on a non-zero status.  Tensors are torch tensors
(device memory and streams come from PyTorch); nothing here computes.
There is no fallback: if the compiled library is missing, importing fails.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libhccs.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_02292_b200.build` "
                      "(needs nvcc); there is no CPU implementation to fall back to")

_lib = ctypes.CDLL(LIB_PATH)

HCCS_OK = 0
HCCS_ERR_INVALID_ARG = 1
HCCS_ERR_CONSTRAINT = 2
HCCS_ERR_NOT_UPLOADED = 3
HCCS_ERR_UNSUPPORTED = 4
HCCS_ERR_CUDA = 5
HCCS_ERR_DEVICE_TIMEOUT = 6

HCCS_OUT_U8 = 0
HCCS_OUT_U16 = 1
HCCS_RECIP_DIV = 0
HCCS_RECIP_CLB = 2
HCCS_CAUSAL = 4

EXPORTS = ("hccs_create", "hccs_destroy", "hccs_params_check", "hccs_params_upload", "hccs_forward",
           "hccs_forward_keylen", "hccs_forward_host",
           "hccs_attention_fused", "hccs_attention_fused_keylen", "hccs_attention_fused_f32", "hccs_attention_fused_i8", "hccs_device_status", "hccs_last_cuda_error", "hccs_status_string",
           "hccs_launch_count", "hccs_forward_static_scratch", "hccs_calibrate", "hccs_debug_wait_timeout")

_vp, _i32, _u32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32

_lib.hccs_create.argtypes = [ctypes.POINTER(_vp), ctypes.c_int]
_lib.hccs_create.restype = ctypes.c_int
_lib.hccs_destroy.argtypes = [_vp]
_lib.hccs_destroy.restype = ctypes.c_int
_lib.hccs_params_upload.argtypes = [_vp, _vp, _i32, _i32, _i32, ctypes.POINTER(_i32), _vp]
_lib.hccs_params_upload.restype = ctypes.c_int
_lib.hccs_params_check.argtypes = [_vp, _i32, _i32, ctypes.POINTER(_i32)]
_lib.hccs_params_check.restype = ctypes.c_int
_lib.hccs_forward.argtypes = [_vp, _vp, _vp, _i32, _i32, _i32, _i32, _u32, _vp]
_lib.hccs_forward.restype = ctypes.c_int
_lib.hccs_forward_keylen.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _u32, _vp]
_lib.hccs_forward_keylen.restype = ctypes.c_int
_lib.hccs_forward_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _u32, _vp]
_lib.hccs_forward_host.restype = ctypes.c_int
_lib.hccs_attention_fused.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                                      _u32, _vp]
_lib.hccs_attention_fused.restype = ctypes.c_int
_lib.hccs_attention_fused_keylen.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                                             _u32, _vp]
_lib.hccs_attention_fused_keylen.restype = ctypes.c_int
_lib.hccs_attention_fused_f32.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32,
                                          _u32, _vp]
_lib.hccs_attention_fused_f32.restype = ctypes.c_int
_lib.hccs_attention_fused_i8.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _i32, _i32, _i32, _i32, _i32,
                                         _u32, _vp]
_lib.hccs_attention_fused_i8.restype = ctypes.c_int
_lib.hccs_device_status.argtypes = [_vp, ctypes.POINTER(_u32), _vp]
_lib.hccs_device_status.restype = ctypes.c_int
_lib.hccs_last_cuda_error.argtypes = [_vp]
_lib.hccs_last_cuda_error.restype = _i32
_lib.hccs_status_string.argtypes = [ctypes.c_int]
_lib.hccs_status_string.restype = ctypes.c_char_p
_lib.hccs_launch_count.argtypes = [_vp]
_lib.hccs_launch_count.restype = ctypes.c_uint64
_lib.hccs_debug_wait_timeout.argtypes = [_vp, _i32, ctypes.c_int64, _vp]
_lib.hccs_debug_wait_timeout.restype = ctypes.c_int


_lib.hccs_forward_static_scratch.argtypes = [_vp, _i32, _i32, _i32, _vp, _vp, _i32, _i32, _i32, _i32, _u32,
                                             ctypes.POINTER(_u32), _vp]
_lib.hccs_forward_static_scratch.restype = ctypes.c_int


class _CalibGrid(ctypes.Structure):
    _fields_ = [(k, _i32) for k in ("D_lo", "D_hi", "D_step", "S_lo", "S_hi", "S_step", "B_step")]


_lib.hccs_calibrate.argtypes = [_vp, _i32, _i32, _i32, _i32, ctypes.c_double, ctypes.POINTER(_CalibGrid), _vp, _vp, _vp]
_lib.hccs_calibrate.restype = ctypes.c_int


def hccs_calibrate(logits, alpha: float, grid, stream=None):
    """Grid-scan calibration of every head on device logits [B,H,Lq,Lk]; grid = (D_lo, D_hi, D_step,
    S_lo, S_hi, S_step, B_step).  Returns (theta int32 [H,3], kl float64 [H])."""
    B, H, Lq, Lk = logits.shape
    _check_tensor(logits, "logits", 1)
    g = _CalibGrid(*[int(v) for v in grid])
    best = np.zeros((H, 3), dtype=np.int32)
    kl = np.zeros(H, dtype=np.float64)
    st = _lib.hccs_calibrate(_ptr(logits), B, H, Lq, Lk, float(alpha), ctypes.byref(g),
                             best.ctypes.data_as(_vp), kl.ctypes.data_as(_vp), _stream_ptr(stream))
    if st != HCCS_OK:
        raise HccsError(st, "hccs_calibrate")
    return best, kl


def hccs_status_string(status: int) -> str:
    return _lib.hccs_status_string(int(status)).decode()


class HccsError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = int(status)
        super().__init__(f"{where}: {hccs_status_string(status)}{(' ' + detail) if detail else ''}")


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return _vp(stream)
    return _vp(stream.cuda_stream)


def _ptr(t):
    return _vp(t.data_ptr()) if t is not None else _vp(0)


def hccs_params_check(params, n_design: int):
    """(status, bad_head) of the host-side admissibility check; needs no GPU."""
    arr = np.ascontiguousarray(params, dtype=np.int32).reshape(-1, 3)
    bad = _i32(-1)
    st = _lib.hccs_params_check(arr.ctypes.data_as(_vp), arr.shape[0], int(n_design), ctypes.byref(bad))
    return int(st), int(bad.value)


class Context:
    """Owns one ``hccs_ctx_t`` (created on ``device``) and exposes the entry points as methods."""

    def __init__(self, device: int = 0):
        h = _vp()
        st = _lib.hccs_create(ctypes.byref(h), int(device))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_create")
        self._h = h
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None):
            _lib.hccs_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- hccs_params_upload
    def hccs_params_upload(self, params, n_design: int, out_shift: int = 0, stream=None) -> None:
        arr = np.ascontiguousarray(params, dtype=np.int32).reshape(-1, 3)
        bad = _i32(-1)
        st = _lib.hccs_params_upload(self._h, arr.ctypes.data_as(_vp), arr.shape[0], int(n_design),
                                     int(out_shift), ctypes.byref(bad), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_params_upload", f"(head {bad.value})" if bad.value >= 0 else "")

    # -- hccs_forward
    def hccs_forward(self, logits, probs, flags: int = 0, stream=None) -> None:
        B, H, Lq, Lk = logits.shape
        _check_tensor(logits, "logits", 1)
        _check_tensor(probs, "probs", 2 if flags & HCCS_OUT_U16 else 1, logits.shape)
        st = _lib.hccs_forward(self._h, _ptr(logits), _ptr(probs), B, H, Lq, Lk, int(flags),
                               _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_forward")

    # -- hccs_forward_keylen
    def hccs_forward_keylen(self, logits, probs, key_len, flags: int = 0, stream=None) -> None:
        B, H, Lq, Lk = logits.shape
        _check_tensor(logits, "logits", 1)
        _check_tensor(probs, "probs", 2 if flags & HCCS_OUT_U16 else 1, logits.shape)
        _check_tensor(key_len, "key_len", 4, (B,))
        st = _lib.hccs_forward_keylen(self._h, _ptr(logits), _ptr(probs), _ptr(key_len), B, H, Lq, Lk,
                                      int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_forward_keylen")

    # -- hccs_forward_host
    def hccs_forward_host(self, logits_host, probs_host, logits_staging, probs_staging,
                          flags: int = 0, stream=None) -> None:
        B, H, Lq, Lk = logits_host.shape
        osz = 2 if flags & HCCS_OUT_U16 else 1
        _check_tensor(logits_host, "logits_host", 1, device="cpu")
        _check_tensor(probs_host, "probs_host", osz, logits_host.shape, device="cpu")
        _check_tensor(logits_staging, "logits_staging", 1, logits_host.shape)
        _check_tensor(probs_staging, "probs_staging", osz, logits_host.shape)
        st = _lib.hccs_forward_host(self._h, _ptr(logits_host), _ptr(probs_host), _ptr(logits_staging),
                                    _ptr(probs_staging), B, H, Lq, Lk, int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_forward_host")

    # -- hccs_attention_fused
    def hccs_attention_fused(self, Q, K, V, O, requant_mult, requant_shift: int, flags: int = 0,
                             stream=None) -> None:
        B, H, L, d = Q.shape
        for name, t in (("Q", Q), ("K", K), ("V", V)):
            _check_tensor(t, name, 1, Q.shape)
        _check_tensor(O, "O", 4, Q.shape)
        mult = np.ascontiguousarray(requant_mult, dtype=np.int32).reshape(-1)
        if mult.size != H:
            raise ValueError("requant_mult must have H entries")
        st = _lib.hccs_attention_fused(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                       mult.ctypes.data_as(_vp), int(requant_shift), B, H, L, d,
                                       int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_attention_fused")

    # -- hccs_attention_fused_keylen
    def hccs_attention_fused_keylen(self, Q, K, V, O, key_len, requant_mult, requant_shift: int,
                                    flags: int = 0, stream=None) -> None:
        B, H, L, d = Q.shape
        for name, t in (("Q", Q), ("K", K), ("V", V)):
            _check_tensor(t, name, 1, Q.shape)
        _check_tensor(O, "O", 4, Q.shape)
        _check_tensor(key_len, "key_len", 4, (B,))
        mult = np.ascontiguousarray(requant_mult, dtype=np.int32).reshape(-1)
        if mult.size != H:
            raise ValueError("requant_mult must have H entries")
        st = _lib.hccs_attention_fused_keylen(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(key_len),
                                              mult.ctypes.data_as(_vp), int(requant_shift), B, H, L, d,
                                              int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_attention_fused_keylen")

    # -- hccs_attention_fused_f32
    def hccs_attention_fused_f32(self, Q, K, V, O, out_scale, requant_mult, requant_shift: int,
                                 flags: int = 0, stream=None) -> None:
        B, H, L, d = Q.shape
        for name, t in (("Q", Q), ("K", K), ("V", V)):
            _check_tensor(t, name, 1, Q.shape)
        _check_tensor(O, "O", 4, Q.shape)
        mult = np.ascontiguousarray(requant_mult, dtype=np.int32).reshape(-1)
        scale = np.ascontiguousarray(out_scale, dtype=np.float32).reshape(-1)
        if mult.size != H or scale.size != H:
            raise ValueError("requant_mult and out_scale must have H entries")
        st = _lib.hccs_attention_fused_f32(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                           scale.ctypes.data_as(_vp), mult.ctypes.data_as(_vp),
                                           int(requant_shift), B, H, L, d, int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_attention_fused_f32")

    # -- hccs_attention_fused_i8
    def hccs_attention_fused_i8(self, Q, K, V, O, out_mult, out_shift: int, requant_mult, requant_shift: int,
                                flags: int = 0, stream=None) -> None:
        B, H, L, d = Q.shape
        for name, t in (("Q", Q), ("K", K), ("V", V)):
            _check_tensor(t, name, 1, Q.shape)
        _check_tensor(O, "O", 1, Q.shape)
        mult = np.ascontiguousarray(requant_mult, dtype=np.int32).reshape(-1)
        omult = np.ascontiguousarray(out_mult, dtype=np.int32).reshape(-1)
        if mult.size != H or omult.size != H:
            raise ValueError("requant_mult and out_mult must have H entries")
        st = _lib.hccs_attention_fused_i8(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), omult.ctypes.data_as(_vp),
                                          int(out_shift), mult.ctypes.data_as(_vp), int(requant_shift), B, H, L, d,
                                          int(flags), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_attention_fused_i8")

    # -- hccs_device_status / hccs_last_cuda_error / hccs_launch_count
    def hccs_device_status(self, stream=None) -> int:
        w = _u32(0)
        st = _lib.hccs_device_status(self._h, ctypes.byref(w), _stream_ptr(stream))
        if st not in (HCCS_OK, HCCS_ERR_DEVICE_TIMEOUT):
            raise HccsError(st, "hccs_device_status")
        return int(w.value)

    # -- hccs_debug_wait_timeout
    def hccs_debug_wait_timeout(self, mode: int, limit_cycles: int, stream=None) -> None:
        st = _lib.hccs_debug_wait_timeout(self._h, int(mode), int(limit_cycles), _stream_ptr(stream))
        if st != HCCS_OK:
            raise HccsError(st, "hccs_debug_wait_timeout")

    def hccs_last_cuda_error(self) -> int:
        return int(_lib.hccs_last_cuda_error(self._h))

    def hccs_launch_count(self) -> int:
        return int(_lib.hccs_launch_count(self._h))


def hccs_forward_static_scratch(params, n_design: int, logits, probs, flags: int = 0, out_shift: int = 0,
                                check_timeout: bool = False, stream=None) -> int:
    """hccs_forward without a context and without any allocation inside the library: for callers
    that may not allocate device memory.  Runs on the current device; ``logits``/``probs`` are the
    caller's tensors.  With ``check_timeout`` the call synchronises and returns the status word."""
    arr = np.ascontiguousarray(params, dtype=np.int32).reshape(-1, 3)
    B, H, Lq, Lk = logits.shape
    _check_tensor(logits, "logits", 1)
    _check_tensor(probs, "probs", 2 if flags & HCCS_OUT_U16 else 1, logits.shape)
    word = _u32(0)
    st = _lib.hccs_forward_static_scratch(arr.ctypes.data_as(_vp), arr.shape[0], int(n_design),
                                          int(out_shift), _ptr(logits), _ptr(probs), B, H, Lq, Lk,
                                          int(flags), ctypes.byref(word) if check_timeout else None,
                                          _stream_ptr(stream))
    if st != HCCS_OK:
        raise HccsError(st, "hccs_forward_static_scratch")
    return int(word.value)


def _check_tensor(t, name, itemsize, shape=None, device="cuda"):
    if t.device.type != device:
        raise ValueError(f"{name} must live on {device}, not {t.device}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if t.element_size() != itemsize:
        raise ValueError(f"{name} must have {itemsize}-byte elements, got {t.dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")


def raw():
    """The underlying ``ctypes.CDLL`` (for tests that call the C ABI with bad arguments)."""
    return _lib
