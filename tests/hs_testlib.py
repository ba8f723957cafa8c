"""Helpers shared by the GPU parity tests: tolerances of the benchmark contract and tensor plumbing."""
import numpy as np
import torch


def to_dev(arr, device="cuda"):
    """numpy storage array (float32, or uint16 bf16 bit patterns, or uint8 signs) -> CUDA tensor."""
    t = torch.from_numpy(np.ascontiguousarray(arr))
    if arr.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device)


def to_f64(t):
    """CUDA tensor of the library's storage types -> numpy float64 (exact widening)."""
    return t.detach().to(torch.float64).cpu().numpy()


def storage_f64(arr):
    if arr.dtype == np.uint16:
        return (arr.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return arr.astype(np.float64)


def tol_positive(log_a64, logx_ref):
    """2e-6 * (1 + |a*_t| + |log(x0 + b*_t)|) + 1e-5, with log(x0 + b*_t) = log x_ref - a*_t (Eq. 1)."""
    astar = np.cumsum(log_a64, axis=1)
    with np.errstate(invalid="ignore"):
        resid = np.abs(logx_ref - astar)
    resid = np.where(np.isfinite(resid), resid, 0.0)
    astar = np.where(np.isfinite(astar), np.abs(astar), 0.0)
    return 2e-6 * (1.0 + astar + resid) + 1e-5


def assert_log_close(got, ref, tol, what=""):
    """Elementwise |got - ref| <= tol; -inf must match exactly."""
    inf_ref = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), inf_ref), f"{what}: -inf pattern differs"
    assert not np.isnan(got).any(), f"{what}: NaN in output"
    err = np.where(inf_ref, 0.0, np.abs(got - np.where(inf_ref, 0.0, ref)))
    bad = err > tol
    if bad.any():
        i = np.unravel_index(np.argmax(err / tol), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} elements over tolerance; worst at {i}: got {got[i]!r} ref {ref[i]!r} "
                             f"err {err[i]:.3e} tol {tol[i]:.3e}")
    return float((err / tol).max())


def assert_signed_close(x_got, x_ref, what=""):
    """|x_gpu - x_ref| <= 1e-3 * max_row |x_ref|."""
    assert not np.isnan(x_got).any(), f"{what}: NaN in output"
    scale = np.abs(x_ref).max(axis=1, keepdims=True)
    err = np.abs(x_got - x_ref)
    tol = 1e-3 * scale
    bad = err > tol
    if bad.any():
        i = np.unravel_index(np.argmax(err - tol), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} elements over tolerance; worst at {i}: got {x_got[i]!r} ref {x_ref[i]!r}")
    return float((err / np.maximum(tol, 1e-300)).max())
