"""The un-fused evaluation of Eq. 7 that `bench.py --ablation unfused` times (framework cumsum and
LogCumSumExp kernels, the way the paper ran the method) against the float64 oracle, at the tolerance of
the positive-input contract, on reduced configurations 2 and 3.  It shows that the ablation compares two
correct evaluations, and it records how close the literal global form comes to the tolerance in fp32."""
import numpy as np
import pytest
import torch

from hs_testlib import assert_log_close, to_dev, to_f64, tol_positive
from paper_2311_06281_b200 import unfused_eq7, workloads

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cid,rows,n", [(2, 512, 2048), (3, 1, 1 << 22)])
def test_unfused_eq7_matches_the_oracle(hs, oracle, cid, rows, n):
    w = workloads.make(cid, rows=rows, n=n)
    t = w.tensors
    out = unfused_eq7.scan_log_unfused(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]))
    torch.cuda.synchronize()
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    tol = tol_positive(t["log_a"].astype(np.float64), ref)
    worst = assert_log_close(to_f64(out), ref, tol, f"unfused Eq. 7, cfg{cid} {rows}x{n}")
    assert worst <= 1.0
    # the fused kernel on the same inputs, same tolerance: both evaluations are correct, so the ablation's
    # timing compares like with like
    ws = hs.new_workspace(rows, n, "cuda")
    fused = hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]), workspace=ws)
    hs.check(ws)
    assert_log_close(to_f64(fused), ref, tol, f"fused, cfg{cid} {rows}x{n}")
