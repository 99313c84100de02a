"""ctypes front end of the plain-C HCCS oracle (``hccs_oracle.c``).

TEST INFRASTRUCTURE, not part of the product: only the tests, the smoke check
and the benchmark's CPU-baseline leg may import this module.  It shares no
code with the CUDA library and never imports it.

The C file holds all the arithmetic (Algorithm 1 and Section III of the paper
in int64).  This module compiles it with gcc on first use, marshals numpy
arrays, and can spread *independent rows* over Python threads (ctypes drops the
GIL during the call); the per-row arithmetic is untouched by that.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hccs_oracle.c")
_LIB = os.path.join(_HERE, "libhccs_oracle.so")

MODE_U16 = 1      # int16 output path, T = 32767 (Eq. 6); otherwise uint8, T = 255 (Eq. 8)
MODE_CLB = 2      # leading-bit reciprocal (Eq. 9) instead of the exact divide
MODE_CAUSAL = 4   # position j of query i valid when j <= i + (Lk - Lq)

_lock = threading.Lock()
_lib = None

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile ``hccs_oracle.c`` into ``libhccs_oracle.so`` beside it (gcc -O2)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared",
                        _SRC, "-o", tmp], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _declare(L: ctypes.CDLL) -> ctypes.CDLL:
    """Argument and result types of every function of the C file."""
    L.hccs_oracle_check_params.argtypes = [_i64] * 4
    L.hccs_oracle_check_params.restype = ctypes.c_int
    L.hccs_oracle_rho.argtypes = [_i64, ctypes.c_int]
    L.hccs_oracle_rho.restype = _i64
    L.hccs_oracle_row.argtypes = [_p, _p, _i64, _i64, _i64, _i64, ctypes.c_int, _i64,
                                  _p, _p, _p]
    L.hccs_oracle_row.restype = _i64
    L.hccs_oracle_forward.argtypes = [_p, _p, _i64, _i64, _i64, _i64, _p, ctypes.c_int,
                                      _i64, _i64, _i64, _p, _p, _p]
    L.hccs_oracle_forward.restype = ctypes.c_int
    L.hccs_oracle_requant.argtypes = [_i64, _i64, _i64]
    L.hccs_oracle_requant.restype = _i64
    L.hccs_oracle_requant_output.argtypes = [_p, _p, _p, _i64, _i64, _i64, _i64, _i64]
    L.hccs_oracle_requant_output.restype = None
    L.hccs_oracle_attention.argtypes = [_p, _p, _p, _p, _p, _i64, _p,
                                        _i64, _i64, _i64, _i64, ctypes.c_int, _i64,
                                        _i64, _i64, _i64, _i64, _p, _p, _p, _p, _p, _p]
    L.hccs_oracle_attention.restype = ctypes.c_int
    return L


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            _lib = _declare(ctypes.CDLL(build()))
    return _lib


def use_library(path):
    """Makes every function of this module call the shared library at ``path`` (None: back to the one
    built from ``hccs_oracle.c``).  For the mutation test only, which plants mistakes in copies of the
    C file and checks that the pins notice."""
    global _lib
    with _lock:
        _lib = None if path is None else _declare(ctypes.CDLL(path))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def check_params(B: int, S: int, D: int, n: int) -> int:
    """Bit mask of violated integer range constraints (0 = admissible)."""
    return int(lib().hccs_oracle_check_params(B, S, D, n))


def rho(Z: int, mode: int) -> int:
    return int(lib().hccs_oracle_rho(Z, mode))


def requant(acc: int, M: int, sh: int) -> int:
    return int(lib().hccs_oracle_requant(acc, M, sh))


def row(x, theta, mode: int = 0, out_shift: int = 0, valid=None):
    """One row of Algorithm 1.  Returns (p_hat int64[n], Z, rho)."""
    x = np.ascontiguousarray(x, dtype=np.int8)
    n = x.shape[0]
    v = None if valid is None else np.ascontiguousarray(valid, dtype=np.uint8)
    p = np.zeros(n, dtype=np.int64)
    Z = _i64(0)
    r = _i64(0)
    B, S, D = (int(t) for t in theta)
    lib().hccs_oracle_row(_ptr(x), _ptr(v), n, B, S, D, mode, out_shift, _ptr(p),
                          ctypes.byref(Z), ctypes.byref(r))
    return p, int(Z.value), int(r.value)


def _params_array(params, H):
    a = np.ascontiguousarray(params, dtype=np.int32).reshape(-1)
    if a.size != 3 * H:
        raise ValueError("params must be H triples (B, S, Dmax)")
    return a


def forward(logits, params, mode: int = 0, out_shift: int = 0, threads: int = 1,
            row_range=None, key_len=None):
    """HCCS over a contiguous int8 [B,H,Lq,Lk] array.  Returns uint8 / uint16, same shape.

    ``threads`` > 1 splits the independent rows over that many Python threads.
    ``row_range=(r0, r1)`` computes only those flat rows (the rest stay zero).
    ``key_len`` (int32 [B]) is the padding mask: key j of batch entry b is valid iff j < key_len[b].
    """
    x = np.ascontiguousarray(logits, dtype=np.int8)
    Bt, H, Lq, Lk = x.shape
    pa = _params_array(params, H)
    out = np.zeros(x.shape, dtype=np.uint16 if (mode & MODE_U16) else np.uint8)
    r0, r1 = (0, Bt * H * Lq) if row_range is None else row_range
    L = lib()
    kl = None if key_len is None else np.ascontiguousarray(key_len, dtype=np.int32)
    if kl is not None and kl.shape != (Bt,):
        raise ValueError("key_len must have one entry per batch entry")

    def work(a, b):
        p_tmp = np.zeros(max(Lk, 1), dtype=np.int64)
        v_tmp = np.zeros(max(Lk, 1), dtype=np.uint8)
        rc = L.hccs_oracle_forward(_ptr(x), _ptr(out), Bt, H, Lq, Lk, _ptr(pa), mode,
                                   out_shift, a, b, _ptr(p_tmp), _ptr(v_tmp), _ptr(kl))
        if rc != 0:
            raise OverflowError("oracle output does not fit the output type")

    _spread(work, r0, r1, threads)
    return out


def attention(Q, K, V, M, sh, params, mode: int = 0, out_shift: int = 0, threads: int = 1,
              bh_range=None, q_range=None, want_intermediates: bool = False, key_len=None):
    """Integer attention Q.K^T -> requant -> HCCS (u8) -> P.V for int8 [B,H,L,d] inputs.

    Returns O int32 [B,H,L,d] (and, if asked, the int8 logits and uint8
    probabilities [B,H,L,L]).  Only slices in ``bh_range`` / rows in ``q_range``
    are computed; the rest stay zero.  ``key_len`` (int32 [B], optional): keys at
    and beyond key_len[b] are padding of batch entry b and take no part.
    """
    Q = np.ascontiguousarray(Q, dtype=np.int8)
    K = np.ascontiguousarray(K, dtype=np.int8)
    V = np.ascontiguousarray(V, dtype=np.int8)
    Bt, H, Lx, d = Q.shape
    pa = _params_array(params, H)
    Ma = np.ascontiguousarray(M, dtype=np.int32)
    kl = None if key_len is None else np.ascontiguousarray(key_len, dtype=np.int32).reshape(Bt)
    O = np.zeros((Bt, H, Lx, d), dtype=np.int32)
    lg = np.zeros((Bt, H, Lx, Lx), dtype=np.int8) if want_intermediates else None
    pr = np.zeros((Bt, H, Lx, Lx), dtype=np.uint8) if want_intermediates else None
    b0, b1 = (0, Bt * H) if bh_range is None else bh_range
    q0, q1 = (0, Lx) if q_range is None else q_range
    L = lib()

    def work(a, b):
        x_tmp = np.zeros(Lx, dtype=np.int8)
        p_tmp = np.zeros(Lx, dtype=np.int64)
        v_tmp = np.zeros(Lx, dtype=np.uint8)
        rc = L.hccs_oracle_attention(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(Ma), sh, _ptr(pa),
                                     Bt, H, Lx, d, mode, out_shift, a, b, q0, q1,
                                     _ptr(x_tmp), _ptr(p_tmp), _ptr(v_tmp), _ptr(lg), _ptr(pr), _ptr(kl))
        if rc != 0:
            raise OverflowError(f"oracle attention failed rc={rc}")

    _spread(work, b0, b1, threads)
    if want_intermediates:
        return O, lg, pr
    return O


def requant_output(O, Mo, sh: int):
    """int8 view of an int32 attention output [B,H,L,d]: every element requantised with its head's
    multiplier Mo[h] and the shift sh by the rule of ``requant``."""
    O = np.ascontiguousarray(O, dtype=np.int32)
    Bt, H, Lx, d = O.shape
    Ma = np.ascontiguousarray(Mo, dtype=np.int32).reshape(H)
    out = np.zeros(O.shape, dtype=np.int8)
    lib().hccs_oracle_requant_output(_ptr(O), _ptr(out), _ptr(Ma), int(sh), Bt * H, H, Lx, d)
    return out


def _spread(work, lo, hi, threads):
    n = hi - lo
    if n <= 0:
        return
    threads = max(1, min(int(threads), n))
    if threads == 1:
        work(lo, hi)
        return
    cuts = [lo + (n * t) // threads for t in range(threads + 1)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        for f in [ex.submit(work, cuts[t], cuts[t + 1]) for t in range(threads)]:
            f.result()
