"""The allocation-free entry point (heinsen_scan_log_static) against the regular one and the oracle.

Some callers of this library cannot allocate device memory at the point where they need a scan
(a plug-in inside another framework's callback, a service with a frozen memory plan).  For them the
library keeps the look-back kernel's scratch in a fixed array of its own.  This test calls that entry
point through the C ABI twice in a row -- the second call finds the array as the first one left it --
and compares both results with heinsen_scan_log on the same inputs and with the float64 oracle, within
the tolerance of the other GPU tests; it checks that the device's free memory does not move across the
calls, and that a problem just over the array's capacity is refused while one just under is accepted.
The file sorts last so that a run that stops at the first failure has already executed every other test.
"""
import numpy as np
import pytest
import torch

from hs_testlib import assert_log_close, to_dev, to_f64, tol_positive
from paper_2311_06281_b200 import workloads

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_regular_entry_point_twice(hs, oracle):
    torch.cuda.synchronize()
    for cid, rows, n in ((3, 1, (1 << 20) + 512), (2, 5, 40000)):
        w = workloads.make(cid, rows=rows, n=n)
        la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
        hs.set_path(hs.PATH_LOOKBACK)
        ws = hs.new_workspace(rows, n, "cuda")
        regular = hs.scan_log(la, lb, lx0, workspace=ws)
        hs.check(ws)
        ref, _ = oracle.scan_log(w.tensors["log_a"], w.tensors["log_b"], w.tensors["log_x0"])
        tol = tol_positive(w.tensors["log_a"].astype(np.float64), ref)
        out = torch.full_like(regular, float("nan"))
        stream = torch.cuda.current_stream().cuda_stream
        # the first call on a device looks up the array's address; take it before watching the memory
        assert hs.lib().heinsen_scan_log_static(la.data_ptr(), lb.data_ptr(), lx0.data_ptr(), out.data_ptr(), rows, n,
                                                stream) == 0
        hs.check_static("cuda")
        # (what the loop below does beside the calls, once before the watched region: torch loads the code of a kernel
        # the first time it runs, and the first copy to the host makes the driver set up its staging memory)
        out.fill_(float("nan"))
        to_f64(out)
        torch.equal(out, regular)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        torch_before = torch.cuda.memory_allocated()
        for call in range(2):
            out.fill_(float("nan"))
            status = hs.lib().heinsen_scan_log_static(la.data_ptr(), lb.data_ptr(), lx0.data_ptr(), out.data_ptr(),
                                                      rows, n, stream)
            assert status == 0, hs.strerror(status)
            hs.check_static("cuda")
            # nothing was taken from the device (cudaMalloc and friends would show here) nor through torch
            assert torch.cuda.mem_get_info()[0] == free_before
            assert torch.cuda.memory_allocated() == torch_before
            # same kernel, same tiles, and the carry between the tiles is composed in a fixed order: the same bits
            assert torch.equal(out, regular), f"call {call}: static and regular entry differ"
            assert_log_close(to_f64(out), ref, tol, f"static scratch, call {call}, cfg{cid}")


def test_static_scratch_entry_point_refuses_what_does_not_fit(hs):
    cap = hs.static_max_elements()
    assert cap >= 1 << 26                                 # the single long sequence of the benchmark fits
    assert hs.workspace_bytes(1, cap) <= 1 << 20 < hs.workspace_bytes(1, cap + 4096)
    a = torch.zeros((1, 16), device="cuda")
    x0 = torch.zeros(1, device="cuda")
    L = hs.lib()
    # Size checks come before anything is launched or read, so status codes alone tell: one element over the
    # capacity is refused ...
    assert L.heinsen_scan_log_static(a.data_ptr(), a.data_ptr(), x0.data_ptr(), a.data_ptr(), 1, cap + 4096, None) == 3
    big_rows = 1 << 20                                    # ... and so are a million rows: far more tiles than the array holds
    status = L.heinsen_scan_log_static(a.data_ptr(), a.data_ptr(), x0.data_ptr(), a.data_ptr(), big_rows, 4096, None)
    assert status == 3 and "workspace" in hs.strerror(status)
    assert L.heinsen_scan_log_static(None, a.data_ptr(), x0.data_ptr(), a.data_ptr(), 1, 16, None) == 1
    assert L.heinsen_scan_log_static(a.data_ptr(), a.data_ptr(), x0.data_ptr(), a.data_ptr(), 0, 16, None) == 0
    torch.cuda.synchronize()


def test_static_scratch_entry_point_accepts_its_full_capacity(hs):
    """One row of exactly the capacity runs (its descriptors fill the array to the last slot)."""
    cap = hs.static_max_elements()
    la = torch.full((1, cap), -1e-6, device="cuda")
    lb = torch.zeros((1, cap), device="cuda")
    lx0 = torch.zeros(1, device="cuda")
    out = torch.empty_like(la)
    status = hs.lib().heinsen_scan_log_static(la.data_ptr(), lb.data_ptr(), lx0.data_ptr(), out.data_ptr(), 1, cap,
                                              torch.cuda.current_stream().cuda_stream)
    assert status == 0, hs.strerror(status)
    hs.check_static("cuda")
    # x_t = a x_{t-1} + 1 with a = exp(-1e-6): x_t -> 1/(1-a) ~ 1e6, monotonically
    # closed form of constant a = exp(-1e-6), b = 1, x0 = 1:  x_t = a^t + (1 - a^t) / (1 - a)
    t = np.arange(cap - 3, cap + 1, dtype=np.float64)
    a_t = np.exp(np.float64(np.float32(-1e-6)) * t)
    expect = np.log(a_t + (1 - a_t) / -np.expm1(np.float64(np.float32(-1e-6))))
    assert np.all(np.abs(out[0, -4:].double().cpu().numpy() - expect) < 1e-3)
    del la, lb, out
    torch.cuda.empty_cache()
