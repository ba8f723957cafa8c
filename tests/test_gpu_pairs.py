"""GPU parity of the linear-domain comparison path (pairs (alpha, beta), no logarithms) against the float64
oracle, and the behaviour that separates it from the log-space path: intermediate values outside fp32's range.
"""
import numpy as np
import pytest
import torch

from hs_testlib import assert_signed_close, to_dev, to_f64
from paper_2311_06281_b200 import workloads

pytestmark = pytest.mark.gpu


def run_pairs(hs, oracle, t, what=""):
    a, b, x0 = to_dev(t["a"]), to_dev(t["b"]), to_dev(t["x0"])
    rows, n = t["a"].shape
    ws = hs.new_workspace(rows, n, "cuda")
    x = hs.scan_linear_pairs(a, b, x0, workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_BATCHED
    ref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    return assert_signed_close(to_f64(x), ref, what)


def test_cfg4_reduced(hs, oracle):
    run_pairs(hs, oracle, workloads.make(4, rows=96).tensors, "pairs cfg4 96 rows")          # several rows per warp
    run_pairs(hs, oracle, workloads.make(4, rows=2400, n=2048).tensors, "pairs cfg4 2400x2048")  # one row per warp


def test_cfg1_single_row(hs, oracle):
    assert run_pairs(hs, oracle, workloads.make(1).tensors, "pairs cfg1") < 0.1


@pytest.mark.parametrize("rows", [1, 3, 149])
@pytest.mark.parametrize("n", [1, 2, 15, 17, 127, 512, 513, 1028, 4100])
def test_odd_shapes(hs, oracle, rows, n):
    run_pairs(hs, oracle, workloads.make(4, rows=rows, n=n, seed=rows * 10007 + n).tensors, f"pairs {rows}x{n}")


def test_rows_on_128_byte_lines_with_partial_last_chunk(hs, oracle):
    # one flat TMA box per chunk; the last chunk of each row is partial and must not touch the next row
    run_pairs(hs, oracle, workloads.make(4, rows=1800, n=1056, seed=5).tensors, "pairs 1800x1056")


def test_unaligned_base_takes_the_plain_load_path(hs, oracle):
    t = workloads.make(4, rows=7, n=1001, seed=3).tensors
    rows, n = t["a"].shape
    big = [torch.zeros(rows * n + 1, dtype=torch.float32, device="cuda") for _ in range(3)]
    a, b, x = (g[1:].view(rows, n) for g in big)
    a.copy_(to_dev(t["a"])); b.copy_(to_dev(t["b"]))
    ws = hs.new_workspace(rows, n, "cuda")
    hs.scan_linear_pairs(a, b, to_dev(t["x0"]), x=x, workspace=ws)
    hs.check(ws)
    assert_signed_close(to_f64(x), oracle.scan_linear(t["a"], t["b"], t["x0"]), "pairs unaligned")


def test_zero_coefficients_reset_the_state(hs, oracle):
    rng = np.random.default_rng(11)
    rows, n = 4, 3000
    a = rng.uniform(0.5, 1.0, (rows, n)).astype(np.float32)
    a[:, ::97] = 0.0
    b = rng.standard_normal((rows, n)).astype(np.float32)
    b[:, 5::13] = 0.0
    t = {"a": a, "b": b, "x0": np.zeros(rows, np.float32)}
    run_pairs(hs, oracle, t, "pairs with a_t = 0")


def test_intermediates_outside_fp32_range_are_lost_here_and_kept_in_log_space(hs, oracle):
    """x falls to 1e-80 and is scaled back to 1: the float64 recurrence and the log-space path return 1, the
    linear-domain pairs lose the value when it leaves fp32's range (the case log space exists for)."""
    n = 9
    a = np.array([[1e-20] * 5 + [1e20] * 4], dtype=np.float32)
    b = np.zeros((1, n), np.float32)
    b[0, 0] = 1.0
    x0 = np.zeros(1, np.float32)
    ref = oracle.scan_linear(a, b, x0)
    # the stored fp32 coefficients are not exactly 1e-20 and 1e20: compare with the oracle's own value
    assert 0.9 < ref[0, -1] < 1.1
    ws = hs.new_workspace(1, n, "cuda")
    x_log = to_f64(hs.scan_linear(to_dev(a), to_dev(b), to_dev(x0), workspace=ws))
    hs.check(ws)
    assert abs(x_log[0, -1] / ref[0, -1] - 1.0) < 1e-4
    x_pairs = to_f64(hs.scan_linear_pairs(to_dev(a), to_dev(b), to_dev(x0), workspace=ws))
    hs.check(ws)
    assert x_pairs[0, 0] == 1.0
    assert x_pairs[0, -1] == 0.0


def test_invalid_arguments(hs):
    a = torch.ones(2, 8, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(hs.HeinsenScanError) as e:
        hs.scan_linear_pairs(a, a, torch.ones(2, device="cuda", dtype=torch.bfloat16))
    assert e.value.status == 1
    z = torch.empty(0, 8, device="cuda")
    assert hs.scan_linear_pairs(z, z, torch.empty(0, device="cuda")).shape == (0, 8)
