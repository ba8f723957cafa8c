"""The allocation-free entry point (heinsen_scan_log_static) against the regular one.

Some callers of this library cannot allocate device memory at the point where they need a scan
(a plug-in inside another framework's callback, a service with a frozen memory plan).  For them the
library keeps the look-back kernel's scratch in a fixed array of its own.  This test calls that entry
point through the C ABI twice in a row -- the second call finds the array as the first one left it --
and compares both results with heinsen_scan_log on the same inputs, within the tolerance of the other
GPU tests; it also checks that an oversized problem is refused.  The file sorts last so that a run
that stops at the first failure has already executed every other test.
"""
import numpy as np
import pytest
import torch

from hs_testlib import to_dev, to_f64, tol_positive
from paper_2311_06281_b200 import workloads

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_regular_entry_point_twice(hs):
    torch.cuda.synchronize()
    for cid, rows, n in ((3, 1, (1 << 20) + 512), (2, 5, 40000)):
        w = workloads.make(cid, rows=rows, n=n)
        la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
        hs.set_path(hs.PATH_LOOKBACK)
        ws = hs.new_workspace(rows, n, "cuda")
        ref = hs.scan_log(la, lb, lx0, workspace=ws)
        hs.check(ws)
        ref64 = to_f64(ref)
        tol = tol_positive(w.tensors["log_a"].astype(np.float64), ref64)
        out = torch.full_like(ref, float("nan"))
        before = torch.cuda.memory_allocated()
        for call in range(2):
            out.fill_(float("nan"))
            status = hs.lib().heinsen_scan_log_static(la.data_ptr(), lb.data_ptr(), lx0.data_ptr(), out.data_ptr(),
                                                      rows, n, torch.cuda.current_stream().cuda_stream)
            assert status == 0, hs.strerror(status)
            hs.check_static("cuda")
            assert torch.cuda.memory_allocated() == before   # nothing was allocated through torch either
            got = to_f64(out)
            err = np.abs(got - ref64)
            assert not np.isnan(got).any()
            assert (err <= 2 * tol).all(), f"call {call}: max err/tol {np.max(err / tol):.3g}"


def test_static_scratch_entry_point_refuses_what_does_not_fit(hs):
    cap = hs.static_max_elements()
    assert cap >= 1 << 26                                 # the single long sequence of the benchmark fits
    a = torch.zeros((1, 16), device="cuda")
    x0 = torch.zeros(1, device="cuda")
    L = hs.lib()
    big_rows = 1 << 20                                    # a million rows: far more tiles than the array holds
    status = L.heinsen_scan_log_static(a.data_ptr(), a.data_ptr(), x0.data_ptr(), a.data_ptr(), big_rows, 4096, None)
    assert status == 3 and "workspace" in hs.strerror(status)
    assert L.heinsen_scan_log_static(None, a.data_ptr(), x0.data_ptr(), a.data_ptr(), 1, 16, None) == 1
    assert L.heinsen_scan_log_static(a.data_ptr(), a.data_ptr(), x0.data_ptr(), a.data_ptr(), 0, 16, None) == 0
    torch.cuda.synchronize()
