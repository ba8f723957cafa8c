"""Run by test_gpu_debug_build.py in a process of its own with HEINSEN_SCAN_LIBRARY pointing at the checked
build (-DHEINSEN_DEBUG): small shapes through every kernel, staging path and storage type, each compared
with the float64 oracle; after every call no index check of the checked build may have fired."""
import os
import sys

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))
sys.path.insert(0, HERE)

from hs_testlib import assert_log_close, assert_signed_close, storage_f64, to_dev, to_f64, tol_positive  # noqa: E402
from oracle import heinsen_oracle as oracle  # noqa: E402
from paper_2311_06281_b200 import heinsen_scan as hs, workloads  # noqa: E402


def no_faults(what):
    f = hs.debug_faults()
    assert f is None, f"{what}: check {f[0]} fired, detail {f[1]:#x}, block {f[2]}, thread {f[3]}"


def offset_copy(t, off):
    buf = torch.empty(t.numel() + 8, dtype=t.dtype, device="cuda")
    v = buf[off:off + t.numel()].view(t.shape)
    v.copy_(t)
    return v


def main():
    oracle.build()
    hs.lib()
    assert hs.debug_build(), "this driver must run on the checked build"
    shapes = [(3, 1), (5, 17), (300, 77), (40, 520), (9, 4100), (2, 70004), (1, 33000 + 3), (150, 1056), (37, 2047)]
    calls = 0
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        hs.set_path(path)
        for rows, n in shapes:
            for off in (0, 1):
                tag = f"path {path} {rows}x{n}+{off}"
                # log domain, fp32 / bf16 / fp32 -> bf16
                w = workloads.make(2, rows=rows, n=n, seed=rows + n)
                t = w.tensors
                ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
                tol = tol_positive(t["log_a"].astype(np.float64), ref)
                la, lb = offset_copy(to_dev(t["log_a"]), off), offset_copy(to_dev(t["log_b"]), off)
                out = hs.scan_log(la, lb, to_dev(t["log_x0"]))
                torch.cuda.synchronize()
                no_faults(tag + " log f32")
                assert_log_close(to_f64(out), ref, tol, tag + " log f32")
                out = hs.scan_log(la, lb, to_dev(t["log_x0"]), out_dtype=torch.bfloat16)
                torch.cuda.synchronize()
                no_faults(tag + " log f32->bf16")
                assert_log_close(to_f64(out), ref, tol + 1e-2 * np.abs(ref), tag + " log f32->bf16")
                w5 = workloads.make(5, rows=rows, n=n, seed=rows + n)
                t5 = w5.tensors
                ref5, _ = oracle.scan_log(t5["log_a"], t5["log_b"], t5["log_x0"])
                out = hs.scan_log(offset_copy(to_dev(t5["log_a"]), off), offset_copy(to_dev(t5["log_b"]), off), to_dev(t5["log_x0"]))
                torch.cuda.synchronize()
                no_faults(tag + " log bf16")
                assert_log_close(to_f64(out), ref5, tol_positive(storage_f64(t5["log_a"]), ref5) + 1e-2 * np.abs(ref5), tag + " bf16")
                # signed linear, pairs, sign tensors, complex
                w4 = workloads.make(4, rows=rows, n=n, seed=rows + n)
                t4 = w4.tensors
                ref4 = oracle.scan_linear(t4["a"], t4["b"], t4["x0"])
                a, b, x0 = offset_copy(to_dev(t4["a"]), off), offset_copy(to_dev(t4["b"]), off), to_dev(t4["x0"])
                x = hs.scan_linear(a, b, x0)
                torch.cuda.synchronize()
                no_faults(tag + " linear")
                assert_signed_close(to_f64(x), ref4, tag + " linear")
                if path == hs.PATH_BATCHED:
                    x = hs.scan_linear_pairs(a, b, x0)
                    torch.cuda.synchronize()
                    no_faults(tag + " pairs")
                    assert_signed_close(to_f64(x), ref4, tag + " pairs")
                with np.errstate(divide="ignore"):
                    mag = {k: np.log(np.abs(t4[k].astype(np.float64))).astype(np.float32) for k in ("a", "b", "x0")}
                sgn = {k: (t4[k] < 0).astype(np.uint8) for k in ("a", "b", "x0")}
                lx, sx = hs.scan_log(offset_copy(to_dev(mag["a"]), off), offset_copy(to_dev(mag["b"]), off), to_dev(mag["x0"]),
                                     sign_a=to_dev(sgn["a"]), sign_b=to_dev(sgn["b"]), sign_x0=to_dev(sgn["x0"]))
                torch.cuda.synchronize()
                no_faults(tag + " sign tensors")
                got = np.exp(to_f64(lx)) * np.where(sx.cpu().numpy() == 1, -1.0, 1.0)
                assert_signed_close(got, ref4, tag + " sign tensors")
                z = {k: (mag[k] + 1j * np.pi * sgn[k]).astype(np.complex64) for k in ("a", "b", "x0")}
                zo = hs.scan_log_complex(offset_copy(torch.from_numpy(z["a"]).cuda(), off),
                                         offset_copy(torch.from_numpy(z["b"]).cuda(), off), torch.from_numpy(z["x0"]).cuda())
                torch.cuda.synchronize()
                no_faults(tag + " complex")
                zz = zo.cpu().numpy()
                got = np.exp(zz.real.astype(np.float64)) * np.where(np.round(zz.imag / np.pi) == 1, -1.0, 1.0)
                assert_signed_close(got, ref4, tag + " complex")
                calls += 8
    hs.set_path(hs.PATH_AUTO)
    print(f"checked build ok: {calls} calls, {hs.launch_count()} launches, no check fired")


if __name__ == "__main__":
    main()
