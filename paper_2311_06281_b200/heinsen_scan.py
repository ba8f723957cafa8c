"""Thin Python binding over the C ABI of libheinsen_scan (argument marshalling only).

Every step of the computation runs in the library's CUDA kernels.  PyTorch is used for
device memory and streams.  There is no CPU fallback: if the library has not been built, or
no CUDA device is present, the calls raise.

Names mirror include/heinsen_scan.h: ``scan_linear`` -> ``heinsen_scan_linear``,
``scan_log`` -> ``heinsen_scan_log``, ``scan_log_host`` -> ``heinsen_scan_log_host``, ...
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# HEINSEN_SCAN_LIBRARY selects another build of the same library (the checked build, libheinsen_scan_debug.so)
LIB_PATH = os.environ.get("HEINSEN_SCAN_LIBRARY") or os.path.join(_HERE, "libheinsen_scan.so")

HS_F32, HS_BF16 = 0, 1
HS_OK = 0
PATH_AUTO, PATH_BATCHED, PATH_LOOKBACK = 0, 1, 2

EXPORTS = [
    "heinsen_scan_linear", "heinsen_scan_log", "heinsen_scan_workspace_bytes", "heinsen_scan_check",
    "heinsen_scan_linear_host", "heinsen_scan_log_host", "heinsen_scan_host_scratch_bytes",
    "heinsen_scan_set_path", "heinsen_scan_tune", "heinsen_scan_debug_config", "heinsen_scan_last_path",
    "heinsen_scan_launch_count", "heinsen_scan_strerror", "heinsen_scan_probe_mufu",
    "heinsen_scan_debug_build", "heinsen_scan_debug_faults", "heinsen_scan_debug_window_ok",
    "heinsen_scan_log_static", "heinsen_scan_check_static", "heinsen_scan_static_max_elements",
    "heinsen_scan_log_complex", "heinsen_scan_complex_workspace_bytes",
    "heinsen_scan_linear_pairs",
]
SHORT_EXPORTS = ["scan_linear", "scan_log"]  # the six/ten-argument forms of the two calls


class HeinsenScanError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"libheinsen_scan status {status}: {message}")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2311_06281_b200.build_ext` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.heinsen_scan_linear.argtypes = [vp, vp, vp, vp, i64, i64, ci, vp, sz, vp]
        L.heinsen_scan_linear.restype = ci
        L.heinsen_scan_linear_pairs.argtypes = [vp, vp, vp, vp, i64, i64, ci, vp, sz, vp]
        L.heinsen_scan_linear_pairs.restype = ci
        L.heinsen_scan_log.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, ci, ci, vp, sz, vp]
        L.heinsen_scan_log.restype = ci
        L.heinsen_scan_workspace_bytes.argtypes = [i64, i64]
        L.heinsen_scan_workspace_bytes.restype = sz
        L.heinsen_scan_check.argtypes = [vp, vp]
        L.heinsen_scan_check.restype = ci
        L.heinsen_scan_linear_host.argtypes = [vp, vp, vp, vp, i64, i64, ci, vp, sz, vp]
        L.heinsen_scan_linear_host.restype = ci
        L.heinsen_scan_log_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, ci, ci, vp, sz, vp]
        L.heinsen_scan_log_host.restype = ci
        L.heinsen_scan_host_scratch_bytes.argtypes = [i64, i64, ci, ci, ci]
        L.heinsen_scan_host_scratch_bytes.restype = sz
        L.heinsen_scan_set_path.argtypes = [ci]
        L.heinsen_scan_set_path.restype = ci
        L.heinsen_scan_tune.argtypes = [ctypes.c_char_p, ci]
        L.heinsen_scan_tune.restype = ci
        u64 = ctypes.c_uint64
        L.heinsen_scan_debug_build.restype = ci
        L.heinsen_scan_debug_faults.argtypes = [ctypes.POINTER(u64)]
        L.heinsen_scan_debug_faults.restype = ci
        L.heinsen_scan_debug_window_ok.argtypes = [u64, u64, u64, u64, u64]
        L.heinsen_scan_debug_window_ok.restype = ci
        L.heinsen_scan_probe_mufu.argtypes = [ci, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.heinsen_scan_probe_mufu.restype = ci
        L.heinsen_scan_debug_config.argtypes = [ctypes.c_uint32, i64]
        L.heinsen_scan_debug_config.restype = ci
        L.heinsen_scan_last_path.restype = ci
        L.heinsen_scan_launch_count.restype = i64
        L.heinsen_scan_log_static.argtypes = [vp, vp, vp, vp, i64, i64, vp]
        L.heinsen_scan_log_static.restype = ci
        L.heinsen_scan_check_static.argtypes = [vp]
        L.heinsen_scan_check_static.restype = ci
        L.heinsen_scan_static_max_elements.restype = sz
        L.heinsen_scan_log_complex.argtypes = [vp, vp, vp, vp, i64, i64, vp, sz, vp]
        L.heinsen_scan_log_complex.restype = ci
        L.heinsen_scan_complex_workspace_bytes.argtypes = [i64, i64]
        L.heinsen_scan_complex_workspace_bytes.restype = sz
        L.scan_linear.argtypes = [vp, vp, vp, vp, i64, i64]
        L.scan_linear.restype = ci
        L.scan_log.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64]
        L.scan_log.restype = ci
        L.heinsen_scan_strerror.argtypes = [ci]
        L.heinsen_scan_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().heinsen_scan_strerror(int(status)).decode()


def _check(status: int):
    if status != HS_OK:
        raise HeinsenScanError(status, strerror(status))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return HS_F32
    if t.dtype == torch.bfloat16:
        return HS_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


class _on_device:
    """Make `device` current for the duration of a call (the library launches on the current device);
    free when it already is."""

    def __init__(self, device):
        self.idx = device.index if device.index is not None else torch.cuda.current_device()
        self.prev = None

    def __enter__(self):
        cur = torch.cuda.current_device()
        if cur != self.idx:
            self.prev = cur
            torch.cuda.set_device(self.idx)

    def __exit__(self, *exc):
        if self.prev is not None:
            torch.cuda.set_device(self.prev)
        return False


def _require(t: torch.Tensor, shape, name: str, cuda: bool = True):
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if cuda and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")


def workspace_bytes(rows: int, n: int) -> int:
    return int(lib().heinsen_scan_workspace_bytes(rows, n))


def new_workspace(rows: int, n: int, device) -> torch.Tensor:
    """Uninitialised device scratch for one call at a time of this shape."""
    nbytes = max(256, workspace_bytes(rows, n))
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def set_path(path: int):
    _check(lib().heinsen_scan_set_path(int(path)))


def tune(name: str, value: int = -1):
    """Set a tuning knob (see heinsen_scan_tune in the header); value < 0 restores its default."""
    _check(lib().heinsen_scan_tune(name.encode(), int(value)))


def debug_build() -> bool:
    """True when the loaded library is the checked build (-DHEINSEN_DEBUG)."""
    return bool(lib().heinsen_scan_debug_build())


def debug_faults():
    """The first failed check of the checked build since the last call, as (code, detail, block, thread), or None."""
    out = (ctypes.c_uint64 * 4)()
    rc = lib().heinsen_scan_debug_faults(out)
    if rc < 0:
        raise HeinsenScanError(4, "heinsen_scan_debug_faults: CUDA error")
    return tuple(int(v) for v in out) if rc else None


def probe_mufu(iterations: int = 4096):
    """(results, seconds) of the register-only ex2/lg2 probe kernel on the current device; synchronous."""
    results, seconds = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().heinsen_scan_probe_mufu(int(iterations), ctypes.byref(results), ctypes.byref(seconds)))
    return results.value, seconds.value


def debug_config(lookback_spin_limit: int = 0, mute_tile: int = -1):
    _check(lib().heinsen_scan_debug_config(int(lookback_spin_limit), int(mute_tile)))


def last_path() -> int:
    return int(lib().heinsen_scan_last_path())


def launch_count() -> int:
    return int(lib().heinsen_scan_launch_count())


def check(workspace: torch.Tensor):
    """Synchronise the current stream and raise if the last call on `workspace` failed on the device."""
    _check(lib().heinsen_scan_check(_ptr(workspace), _stream_ptr(workspace.device)))


def scan_linear(a: torch.Tensor, b: torch.Tensor, x0: torch.Tensor, x: torch.Tensor | None = None,
                workspace: torch.Tensor | None = None) -> torch.Tensor:
    """x[r,t] = a[r,t]*x[r,t-1] + b[r,t]; a, b: [rows,n] float32 CUDA; x0: [rows].  Asynchronous."""
    rows, n = a.shape
    _require(a, (rows, n), "a"); _require(b, (rows, n), "b"); _require(x0, (rows,), "x0")
    if x is None:
        x = torch.empty_like(a)
    _require(x, (rows, n), "x")
    if not (a.dtype == b.dtype == x0.dtype == x.dtype):
        raise TypeError("a, b, x0, x must share one dtype")
    if rows == 0 or n == 0:
        return x
    if workspace is None:
        workspace = new_workspace(rows, n, a.device)
    with _on_device(a.device):
        _check(lib().heinsen_scan_linear(_ptr(a), _ptr(b), _ptr(x0), _ptr(x), rows, n, _dtype_code(a),
                                         _ptr(workspace), workspace.numel(), _stream_ptr(a.device)))
    return x


def scan_linear_pairs(a: torch.Tensor, b: torch.Tensor, x0: torch.Tensor, x: torch.Tensor | None = None,
                      workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Comparison path: the same recurrence scanned in the linear domain as (alpha, beta) pairs, no logarithms.
    Arguments as for scan_linear.  Asynchronous."""
    rows, n = a.shape
    _require(a, (rows, n), "a"); _require(b, (rows, n), "b"); _require(x0, (rows,), "x0")
    if x is None:
        x = torch.empty_like(a)
    _require(x, (rows, n), "x")
    if not (a.dtype == b.dtype == x0.dtype == x.dtype):
        raise TypeError("a, b, x0, x must share one dtype")
    if rows == 0 or n == 0:
        return x
    if workspace is None:
        workspace = new_workspace(rows, n, a.device)
    with _on_device(a.device):
        _check(lib().heinsen_scan_linear_pairs(_ptr(a), _ptr(b), _ptr(x0), _ptr(x), rows, n, _dtype_code(a),
                                               _ptr(workspace), workspace.numel(), _stream_ptr(a.device)))
    return x


def scan_log(log_a: torch.Tensor, log_b: torch.Tensor, log_x0: torch.Tensor, log_x: torch.Tensor | None = None,
             sign_a: torch.Tensor | None = None, sign_b: torch.Tensor | None = None,
             sign_x0: torch.Tensor | None = None, sign_x: torch.Tensor | None = None,
             out_dtype: torch.dtype | None = None, workspace: torch.Tensor | None = None):
    """log-domain scan.  Returns log_x, or (log_x, sign_x) when any sign tensor is given.  Asynchronous."""
    rows, n = log_a.shape
    _require(log_a, (rows, n), "log_a"); _require(log_b, (rows, n), "log_b"); _require(log_x0, (rows,), "log_x0")
    if not (log_a.dtype == log_b.dtype == log_x0.dtype):
        raise TypeError("log_a, log_b, log_x0 must share one dtype")
    if log_x is None:
        log_x = torch.empty((rows, n), dtype=out_dtype or log_a.dtype, device=log_a.device)
    _require(log_x, (rows, n), "log_x")
    signed = any(s is not None for s in (sign_a, sign_b, sign_x0))
    for s, shape, name in ((sign_a, (rows, n), "sign_a"), (sign_b, (rows, n), "sign_b"), (sign_x0, (rows,), "sign_x0")):
        if s is not None:
            _require(s, shape, name)
            if s.dtype != torch.uint8:
                raise TypeError(f"{name} must be uint8")
    if signed:
        if sign_x is None:
            sign_x = torch.empty((rows, n), dtype=torch.uint8, device=log_a.device)
        _require(sign_x, (rows, n), "sign_x")
    if rows == 0 or n == 0:
        return (log_x, sign_x) if signed else log_x
    if workspace is None:
        workspace = new_workspace(rows, n, log_a.device)
    with _on_device(log_a.device):
        _check(lib().heinsen_scan_log(_ptr(log_a), _ptr(log_b), _ptr(log_x0), _ptr(log_x), _ptr(sign_a), _ptr(sign_b),
                                      _ptr(sign_x0), _ptr(sign_x) if signed else None, rows, n, _dtype_code(log_a),
                                      _dtype_code(log_x), _ptr(workspace), workspace.numel(),
                                      _stream_ptr(log_a.device)))
    return (log_x, sign_x) if signed else log_x


def scan_log_static(log_a: torch.Tensor, log_b: torch.Tensor, log_x0: torch.Tensor,
                    log_x: torch.Tensor | None = None) -> torch.Tensor:
    """heinsen_scan_log_static: float32 log-domain scan that takes its scratch from a fixed array inside
    the library instead of a caller-provided workspace, for callers that cannot allocate device memory
    (they still pass inputs and the output).  Problems whose descriptors do not fit that array raise
    HeinsenScanError(HS_ERR_WORKSPACE_TOO_SMALL).  Calls must not overlap on the GPU.  Asynchronous."""
    rows, n = log_a.shape
    _require(log_a, (rows, n), "log_a"); _require(log_b, (rows, n), "log_b"); _require(log_x0, (rows,), "log_x0")
    if not (log_a.dtype == log_b.dtype == log_x0.dtype == torch.float32):
        raise TypeError("scan_log_static takes float32 tensors")
    if log_x is None:
        log_x = torch.empty_like(log_a)
    _require(log_x, (rows, n), "log_x")
    if log_x.dtype != torch.float32:
        raise TypeError("scan_log_static writes float32")
    with _on_device(log_a.device):
        _check(lib().heinsen_scan_log_static(_ptr(log_a), _ptr(log_b), _ptr(log_x0), _ptr(log_x), rows, n,
                                             _stream_ptr(log_a.device)))
    return log_x


def check_static(device):
    """Synchronise the current stream of `device` and raise if the last scan_log_static call failed on the device."""
    device = torch.device(device)
    with _on_device(device):
        _check(lib().heinsen_scan_check_static(_stream_ptr(device)))


def static_max_elements() -> int:
    return int(lib().heinsen_scan_static_max_elements())


def scan_log_complex(log_a: torch.Tensor, log_b: torch.Tensor, log_x0: torch.Tensor,
                     log_x: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """heinsen_scan_log_complex: complex64 tensors (log|v| + i*k*pi, k odd for negative v) in and out.  Asynchronous."""
    rows, n = log_a.shape
    _require(log_a, (rows, n), "log_a"); _require(log_b, (rows, n), "log_b"); _require(log_x0, (rows,), "log_x0")
    if not (log_a.dtype == log_b.dtype == log_x0.dtype == torch.complex64):
        raise TypeError("scan_log_complex takes complex64 tensors")
    if log_x is None:
        log_x = torch.empty_like(log_a)
    _require(log_x, (rows, n), "log_x")
    if rows == 0 or n == 0:
        return log_x
    if workspace is None:
        workspace = torch.empty(int(lib().heinsen_scan_complex_workspace_bytes(rows, n)), dtype=torch.uint8,
                                device=log_a.device)
    with _on_device(log_a.device):
        _check(lib().heinsen_scan_log_complex(_ptr(log_a), _ptr(log_b), _ptr(log_x0), _ptr(log_x), rows, n,
                                              _ptr(workspace), workspace.numel(), _stream_ptr(log_a.device)))
    return log_x


def host_scratch_bytes(rows: int, n: int, dtype_in: torch.dtype, dtype_out: torch.dtype, with_signs: bool) -> int:
    code = {torch.float32: HS_F32, torch.bfloat16: HS_BF16}
    return int(lib().heinsen_scan_host_scratch_bytes(rows, n, code[dtype_in], code[dtype_out], int(with_signs)))


def scan_log_host(log_a, log_b, log_x0, log_x, device_scratch: torch.Tensor, sign_a=None, sign_b=None, sign_x0=None,
                  sign_x=None):
    """Host-buffer variant: all tensors are CPU tensors (pinned recommended); synchronous."""
    rows, n = log_a.shape
    for t, shape, name in ((log_a, (rows, n), "log_a"), (log_b, (rows, n), "log_b"), (log_x0, (rows,), "log_x0"),
                           (log_x, (rows, n), "log_x")):
        _require(t, shape, name, cuda=False)
        if t.is_cuda:
            raise ValueError(f"{name} must be a host tensor")
    dev = device_scratch.device
    with _on_device(dev):
        _check(lib().heinsen_scan_log_host(_ptr(log_a), _ptr(log_b), _ptr(log_x0), _ptr(log_x), _ptr(sign_a),
                                           _ptr(sign_b), _ptr(sign_x0), _ptr(sign_x), rows, n, _dtype_code(log_a),
                                           _dtype_code(log_x), _ptr(device_scratch), device_scratch.numel(),
                                           _stream_ptr(dev)))
    return log_x


def scan_linear_host(a, b, x0, x, device_scratch: torch.Tensor):
    """Host-buffer variant of scan_linear: CPU tensors in and out; synchronous."""
    rows, n = a.shape
    for t, shape, name in ((a, (rows, n), "a"), (b, (rows, n), "b"), (x0, (rows,), "x0"), (x, (rows, n), "x")):
        _require(t, shape, name, cuda=False)
        if t.is_cuda:
            raise ValueError(f"{name} must be a host tensor")
    dev = device_scratch.device
    with _on_device(dev):
        _check(lib().heinsen_scan_linear_host(_ptr(a), _ptr(b), _ptr(x0), _ptr(x), rows, n, _dtype_code(a),
                                              _ptr(device_scratch), device_scratch.numel(), _stream_ptr(dev)))
    return x
