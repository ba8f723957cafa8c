"""The largest sizes the library accepts, checked on sampled outputs against closed forms of the recurrence
(the float64 oracle cannot hold these inputs; constant coefficients give x_t = a^t x_0 + b (1 - a^t) / (1 - a)).
Each case holds about 26 GB on the device for a few milliseconds of work.
"""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MAX_N = (1 << 31) - (1 << 20)   # largest n the library accepts
MAX_ROWS = (1 << 31) - 1        # largest row count


def closed_form_log_x(t, log_a, log_b, log_x0):
    """log x_t for constant a in (0,1), b > 0, in float64: log(a^t x0 + b (1 - a^t) / (1 - a))."""
    t = np.asarray(t, dtype=np.float64)
    la_t = t * log_a
    first = la_t + log_x0
    second = log_b + np.log(-np.expm1(la_t)) - math.log(-math.expm1(log_a))
    return np.logaddexp(first, second)


def need_memory(nbytes):
    free, _ = torch.cuda.mem_get_info()
    if free < nbytes:
        pytest.skip(f"needs {nbytes >> 30} GiB of device memory")


def test_one_row_of_the_largest_length(hs):
    need_memory(30 << 30)
    n = MAX_N
    log_a, log_b, log_x0 = math.log(0.999), math.log(0.5), math.log(3.0)
    la = torch.full((1, n), log_a, device="cuda")
    lb = torch.full((1, n), log_b, device="cuda")
    # the fp32 values actually stored decide the expected result
    log_a32, log_b32 = float(la[0, 0].double()), float(lb[0, 0].double())
    x0 = torch.full((1,), log_x0, device="cuda")
    log_x032 = float(x0[0].double())
    ws = hs.new_workspace(1, n, "cuda")
    out = hs.scan_log(la, lb, x0, workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_LOOKBACK
    rng = np.random.default_rng(0)
    idx = np.unique(np.concatenate([np.arange(0, 40), np.arange(n - 40, n), rng.integers(0, n, 4000),
                                    np.arange(1, 300) * 7168 - 1, np.arange(1, 300) * 7168,   # tile edges
                                    n - 1 - np.arange(1, 200) * 512]))                          # chunk edges near the end
    got = out[0, torch.from_numpy(idx).cuda()].double().cpu().numpy()
    ref = closed_form_log_x(idx + 1, log_a32, log_b32, log_x032)
    # the values settle at log(b / (1 - a)) = 6.2; the segment-local evaluation keeps the error near fp32 rounding
    assert np.abs(got - ref).max() < 2e-5, np.abs(got - ref).max()
    assert torch.isfinite(out).all()


def test_the_largest_number_of_rows(hs):
    need_memory(30 << 30)
    rows, n = MAX_ROWS, 1
    a = torch.full((rows, n), 0.5, device="cuda")
    b = torch.empty((rows, n), device="cuda")
    b.copy_((torch.arange(rows, device="cuda") % 1024).float().view(rows, 1))
    x0 = torch.full((rows,), 2.0, device="cuda")
    ws = hs.new_workspace(rows, n, "cuda")
    x = hs.scan_linear(a, b, x0, workspace=ws)
    hs.check(ws)
    assert hs.last_path() == hs.PATH_BATCHED
    expect = 1.0 + (torch.arange(rows, device="cuda") % 1024).float()
    err = (x.view(-1) - expect).abs()
    assert float(err.max()) <= 1e-3 * 1024.0


def test_sizes_beyond_the_limits_are_refused(hs):
    L = hs.lib()
    t = torch.zeros(16, device="cuda")
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = t.data_ptr()
    assert L.heinsen_scan_linear(p, p, p, p, 1, MAX_N + 1, 0, ws.data_ptr(), ws.numel(), None) == 1
    assert L.heinsen_scan_linear(p, p, p, p, MAX_ROWS + 1, 1, 0, ws.data_ptr(), ws.numel(), None) == 1
    assert L.heinsen_scan_workspace_bytes(1, MAX_N + 1) == 0
    assert L.heinsen_scan_workspace_bytes(1, MAX_N) > 0
