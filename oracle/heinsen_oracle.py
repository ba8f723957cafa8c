"""ctypes loader for the float64 CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It shares nothing with the CUDA path: its arithmetic lives in
``heinsen_oracle.c`` (the sequential recurrence of the paper's Abstract and
Proof section, Eq. 4) and is compiled here with plain gcc.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "heinsen_oracle.c")
_LIB = os.path.join(_HERE, "libheinsen_oracle.so")

F32, BF16, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math) if it is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.oracle_max_threads.restype = ci
        lib.oracle_scan_linear.argtypes = [vp, vp, vp, vp, i64, i64, ci, ci]
        lib.oracle_scan_linear.restype = None
        lib.oracle_scan_log.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, ci, ci]
        lib.oracle_scan_log.restype = None
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _storage(arr, shape):
    """Return (contiguous array, dtype code).  bf16 storage is passed as uint16 bit patterns."""
    arr = np.ascontiguousarray(arr)
    if arr.shape != shape:
        raise ValueError(f"expected shape {shape}, got {arr.shape}")
    if arr.dtype == np.float32:
        return arr, F32
    if arr.dtype == np.uint16:
        return arr, BF16
    if arr.dtype == np.float64:
        return arr, F64
    raise TypeError(f"unsupported storage dtype {arr.dtype}")


def _ptr(arr):
    return None if arr is None else arr.ctypes.data_as(ctypes.c_void_p)


def scan_linear(a, b, x0, nthreads: int | None = None) -> np.ndarray:
    """x[r,t] = a[r,t]*x[r,t-1] + b[r,t] in float64; a, b: [rows,n]; x0: [rows]."""
    a = np.asarray(a)
    rows, n = a.shape
    a, dt = _storage(a, (rows, n))
    b, dtb = _storage(b, (rows, n))
    x0, dt0 = _storage(x0, (rows,))
    if not (dt == dtb == dt0):
        raise TypeError("a, b, x0 must share one storage dtype")
    x = np.empty((rows, n), dtype=np.float64)
    nt = max_threads() if nthreads is None else int(nthreads)
    _load().oracle_scan_linear(_ptr(a), _ptr(b), _ptr(x0), _ptr(x), rows, n, dt, nt)
    return x


def scan_log(log_a, log_b, log_x0, sign_a=None, sign_b=None, sign_x0=None,
             nthreads: int | None = None):
    """Sign+magnitude log-domain recurrence in float64.

    Returns (log|x| float64 [rows,n], sign uint8 [rows,n]); sign 1 = negative.
    """
    log_a = np.asarray(log_a)
    rows, n = log_a.shape
    log_a, dt = _storage(log_a, (rows, n))
    log_b, dtb = _storage(log_b, (rows, n))
    log_x0, dt0 = _storage(log_x0, (rows,))
    if not (dt == dtb == dt0):
        raise TypeError("log_a, log_b, log_x0 must share one storage dtype")

    def sg(s, shape):
        if s is None:
            return None
        s = np.ascontiguousarray(s, dtype=np.uint8)
        if s.shape != shape:
            raise ValueError("sign tensor shape mismatch")
        return s

    sign_a, sign_b, sign_x0 = sg(sign_a, (rows, n)), sg(sign_b, (rows, n)), sg(sign_x0, (rows,))
    log_x = np.empty((rows, n), dtype=np.float64)
    sign_x = np.empty((rows, n), dtype=np.uint8)
    nt = max_threads() if nthreads is None else int(nthreads)
    _load().oracle_scan_log(_ptr(log_a), _ptr(log_b), _ptr(log_x0), _ptr(sign_a), _ptr(sign_b),
                            _ptr(sign_x0), _ptr(log_x), _ptr(sign_x), rows, n, dt, nt)
    return log_x, sign_x
