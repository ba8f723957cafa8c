"""The five benchmark configurations at their full sizes, in the launch configuration bench.py times
(automatic kernel selection), against the float64 oracle: element by element where the oracle finishes
in seconds (configurations 1-4), on sampled rows plus a full-size recurrence-residual property for
configuration 5 (2^29 elements)."""
import numpy as np
import pytest
import torch

from hs_testlib import assert_log_close, assert_signed_close, storage_f64, to_dev, to_f64, tol_positive
from paper_2311_06281_b200 import workloads

pytestmark = pytest.mark.gpu


def test_cfg2_full_size(hs, oracle):
    w = workloads.make(2)
    t = w.tensors
    ws = hs.new_workspace(w.rows, w.n, "cuda")
    out = hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]), workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_BATCHED
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    worst = assert_log_close(to_f64(out), ref, tol_positive(t["log_a"].astype(np.float64), ref), "cfg2 full")
    assert worst < 0.5


def test_cfg3_full_size_log_and_linear(hs, oracle):
    w = workloads.make(3)
    t = w.tensors
    ws = hs.new_workspace(w.rows, w.n, "cuda")
    out = hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]), workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_LOOKBACK
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    assert_log_close(to_f64(out), ref, tol_positive(t["log_a"].astype(np.float64), ref), "cfg3 log full")
    del out
    # secondary: the linear entry point on a = fp32(exp(log_a)), b, x0 = 0.5
    x = hs.scan_linear(to_dev(t["a"]), to_dev(t["b"]), to_dev(t["x0"]), workspace=ws)
    hs.check(ws)
    xref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    logref = np.log(xref)
    tol = tol_positive(np.log(t["a"].astype(np.float64)), logref)
    got = to_f64(x)
    assert (got > 0).all()
    assert_log_close(np.log(got), logref, tol, "cfg3 linear full")


def test_cfg4_full_size_signed(hs, oracle):
    w = workloads.make(4)
    t = w.tensors
    ws = hs.new_workspace(w.rows, w.n, "cuda")
    x = hs.scan_linear(to_dev(t["a"]), to_dev(t["b"]), to_dev(t["x0"]), workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_BATCHED
    ref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    got = to_f64(x)
    assert_signed_close(got, ref, "cfg4 full")
    # x stays real under signed inputs: finite, and both signs occur
    assert np.isfinite(got).all() and (got < 0).any() and (got > 0).any()


def test_cfg5_full_size_bf16_sampled_rows_and_residual(hs, oracle):
    w = workloads.make(5)
    t = w.tensors
    la, lb, lx0 = to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"])
    ws = hs.new_workspace(w.rows, w.n, "cuda")
    out = hs.scan_log(la, lb, lx0, workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_BATCHED and out.dtype == torch.bfloat16
    rng = np.random.default_rng(5)
    rows = sorted(set([0, 1, 147, 148, 149, 2367, 2368, 16383, 16384, w.rows - 2, w.rows - 1] +
                      list(rng.integers(0, w.rows, 53))))
    sub = {k: np.ascontiguousarray(v[rows]) for k, v in t.items()}
    ref, _ = oracle.scan_log(sub["log_a"], sub["log_b"], sub["log_x0"])
    got = to_f64(out[torch.tensor(rows, device="cuda")])
    tol = tol_positive(storage_f64(sub["log_a"]), ref) + 1e-2 * np.abs(ref)
    assert_log_close(got, ref, tol, "cfg5 sampled rows")
    # every element, in float64 on the device: log x_t = logaddexp(log a_t + log x_{t-1}, log b_t) up to the
    # bf16 rounding of the two stored outputs it involves
    worst = 0.0
    for r0 in range(0, w.rows, 2048):
        sl = slice(r0, r0 + 2048)
        y = out[sl].double()
        prev = torch.cat([lx0[sl].double()[:, None], y[:, :-1]], dim=1)
        pred = torch.logaddexp(la[sl].double() + prev, lb[sl].double())
        bound = 2.0 ** -8 * (y.abs() + prev.abs()) + 1e-4
        worst = max(worst, float(((y - pred).abs() / bound).max()))
    assert worst <= 1.0, worst


def test_cfg1_full_size(hs, oracle):
    w = workloads.make(1)
    t = w.tensors
    x = hs.scan_linear(to_dev(t["a"]), to_dev(t["b"]), to_dev(t["x0"]))
    ref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    logref = np.log(ref)
    assert_log_close(np.log(to_f64(x)), logref, tol_positive(np.log(t["a"].astype(np.float64)), logref), "cfg1")
