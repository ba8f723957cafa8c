"""GPU parity: the CUDA path, called through the C ABI, against the float64 CPU oracle on identical
seeded inputs.  Tolerances are the benchmark contract's:
  positive inputs : |log x_gpu - log x_ref| <= 2e-6 (1 + |a*_t| + |log(x0 + b*_t)|) + 1e-5
  signed inputs   : |x_gpu - x_ref| <= 1e-3 max_row |x_ref|
  bf16 storage    : relative error of the stored log x <= 1e-2 (+ the fp32 tolerance as floor)
"""
import numpy as np
import pytest
import torch

from hs_testlib import assert_log_close, assert_signed_close, storage_f64, to_dev, to_f64, tol_positive
from paper_2311_06281_b200 import workloads

pytestmark = pytest.mark.gpu


def run_log(hs, oracle, t, path=None, signs=None, out_dtype=None, what=""):
    """scan_log on the GPU vs oracle.scan_log; positive-input tolerance (bf16 tolerance if stored as bf16)."""
    if path is not None:
        hs.set_path(path)
    la, lb, lx0 = to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"])
    rows, n = t["log_a"].shape
    ws = hs.new_workspace(rows, n, "cuda")
    out = hs.scan_log(la, lb, lx0, out_dtype=out_dtype, workspace=ws)
    hs.check(ws)
    got = to_f64(out)
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    tol = tol_positive(storage_f64(t["log_a"]), ref)
    if out.dtype == torch.bfloat16:
        tol = tol + 1e-2 * np.abs(np.where(np.isfinite(ref), ref, 0.0))
    return assert_log_close(got, ref, tol, what)


def run_linear(hs, oracle, t, path=None, signed=False, what=""):
    if path is not None:
        hs.set_path(path)
    a, b, x0 = to_dev(t["a"]), to_dev(t["b"]), to_dev(t["x0"])
    rows, n = t["a"].shape
    ws = hs.new_workspace(rows, n, "cuda")
    x = hs.scan_linear(a, b, x0, workspace=ws)
    hs.check(ws)
    got = to_f64(x)
    ref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    if signed:
        return assert_signed_close(got, ref, what)
    assert (got > 0).all(), f"{what}: non-positive output for positive inputs"
    logref = np.log(ref)
    with np.errstate(divide="ignore"):
        tol = tol_positive(np.log(t["a"].astype(np.float64)), logref)
    return assert_log_close(np.log(got), logref, tol, what)


# ------------------------------------------------------------------------------------------ configs, reduced
def test_cfg1_single_sequence_linear(hs, oracle):
    w = workloads.make(1)
    r = run_linear(hs, oracle, w.tensors, what="cfg1")
    assert hs.last_path() == hs.PATH_LOOKBACK
    assert r < 1.0
    run_linear(hs, oracle, w.tensors, path=hs.PATH_BATCHED, what="cfg1 batched")


def test_cfg1_closed_form_constant_ab(hs):
    # x_t = 10 - 9*0.95^t for a = 0.95, b = 0.5, x0 = 1, from the stored fp32 value of 0.95
    n = 4096
    a32 = np.float32(0.95)
    t = np.arange(1, n + 1, dtype=np.float64)
    af = float(a32)
    ref = af ** t + 0.5 * (1 - af ** t) / (1 - af)
    for path in (hs.PATH_LOOKBACK, hs.PATH_BATCHED):
        hs.set_path(path)
        x = hs.scan_linear(torch.full((1, n), 0.95, device="cuda"), torch.full((1, n), 0.5, device="cuda"),
                           torch.ones(1, device="cuda"))
        got = to_f64(x)[0]
        tol = 2e-6 * (1 + np.abs(t * np.log(af)) + np.abs(np.log(ref) - t * np.log(af))) + 1e-5
        assert (np.abs(np.log(got) - np.log(ref)) <= tol).all()


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_cfg2_reduced(hs, oracle, path):
    w = workloads.make(2, rows=1500)
    r = run_log(hs, oracle, w.tensors, path=getattr(hs, "PATH_" + path.upper()), what=f"cfg2/{path}")
    assert r < 1.0


@pytest.mark.parametrize("n", [(1 << 20) + 76, (1 << 18) + 3])  # TMA with ragged tail; unaligned pitch
def test_cfg3_reduced_long_sequence(hs, oracle, n):
    w = workloads.make(3, rows=1, n=n)
    run_log(hs, oracle, w.tensors, what=f"cfg3 log n={n}")
    assert hs.last_path() == hs.PATH_LOOKBACK
    run_linear(hs, oracle, w.tensors, what=f"cfg3 linear n={n}")


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_cfg4_reduced_signed_linear(hs, oracle, path):
    w = workloads.make(4, rows=96)
    run_linear(hs, oracle, w.tensors, path=getattr(hs, "PATH_" + path.upper()), signed=True, what=f"cfg4/{path}")


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_cfg4_reduced_signed_log_with_sign_tensors(hs, oracle, path):
    w = workloads.make(4, rows=64, n=4096)
    t = w.tensors
    a64, b64, x064 = (t[k].astype(np.float64) for k in ("a", "b", "x0"))
    la = np.log(np.abs(a64)).astype(np.float32)
    lb = np.log(np.abs(b64)).astype(np.float32)
    lx0 = np.log(np.abs(x064)).astype(np.float32)
    sa, sb, sx0 = (a64 < 0).astype(np.uint8), (b64 < 0).astype(np.uint8), (x064 < 0).astype(np.uint8)
    hs.set_path(getattr(hs, "PATH_" + path.upper()))
    lx, sx = hs.scan_log(to_dev(la), to_dev(lb), to_dev(lx0), sign_a=to_dev(sa), sign_b=to_dev(sb), sign_x0=to_dev(sx0))
    ref_l, ref_s = oracle.scan_log(la, lb, lx0, sa, sb, sx0)
    got = np.where(sx.cpu().numpy() == 1, -1.0, 1.0) * np.exp(to_f64(lx))
    ref = np.where(ref_s == 1, -1.0, 1.0) * np.exp(ref_l)
    assert set(np.unique(sx.cpu().numpy())) <= {0, 1}
    assert_signed_close(got, ref, f"cfg4 log+signs/{path}")


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_cfg5_reduced_bf16(hs, oracle, path):
    w = workloads.make(5, rows=1300 if path == "batched" else 40)
    run_log(hs, oracle, w.tensors, path=getattr(hs, "PATH_" + path.upper()), what=f"cfg5/{path}")


def test_f32_in_bf16_out(hs, oracle):
    w = workloads.make(2, rows=1300, n=1024)
    run_log(hs, oracle, w.tensors, out_dtype=torch.bfloat16, what="f32->bf16")


# ------------------------------------------------------------------------------------------ shapes
@pytest.mark.parametrize("rows", [1, 3, 149])
@pytest.mark.parametrize("n", [1, 2, 3, 5, 15, 16, 17, 31, 33, 127, 511, 512, 513, 1028, 4100, 8195])
def test_odd_shapes_both_paths(hs, oracle, rows, n):
    w = workloads.make(2, rows=rows, n=n, seed=rows * 100003 + n)
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        run_log(hs, oracle, w.tensors, path=path, what=f"{rows}x{n}/{path}")


@pytest.mark.parametrize("rows,n", [(40000, 77), (30001, 160), (12000, 1536), (70000, 33)])
def test_many_rows_handed_out_by_tickets(hs, oracle, rows, n):
    """Enough row groups per warp slot for the batched kernel to draw them from its ticket counter: several rows
    per warp without TMA (n*4 % 16 != 0), several rows per warp with TMA boxes, one row per warp with flat boxes."""
    w = workloads.make(2, rows=rows, n=n, seed=rows + n)
    run_log(hs, oracle, w.tensors, path=hs.PATH_BATCHED, what=f"tickets {rows}x{n}")
    # twice on the same workspace: the second call must take over the first call's ticket word
    la, lb, lx0 = to_dev(w.tensors["log_a"]), to_dev(w.tensors["log_b"]), to_dev(w.tensors["log_x0"])
    ws = hs.new_workspace(rows, n, "cuda")
    first = hs.scan_log(la, lb, lx0, workspace=ws)
    second = hs.scan_log(la, lb, lx0, workspace=ws)
    hs.check(ws)
    assert torch.equal(first, second)


@pytest.mark.parametrize("rows,n,cid", [(50000, 16, 2), (40000, 24, 2), (30011, 32, 2), (30000, 40, 2), (25000, 64, 2),
                                         (20000, 100, 2), (20000, 128, 2), (30000, 48, 5), (30000, 40, 4)])
def test_many_short_rows(hs, oracle, rows, n, cid):
    """Rows shorter than a chunk: the warp holds 2 to 16 rows, chosen so that the chunks pad the rows least."""
    w = workloads.make(cid, rows=rows, n=n, seed=rows + n)
    if cid == 4:
        run_linear(hs, oracle, w.tensors, path=hs.PATH_BATCHED, signed=True, what=f"short rows {rows}x{n}")
    else:
        run_log(hs, oracle, w.tensors, path=hs.PATH_BATCHED, what=f"short rows {rows}x{n}")


@pytest.mark.parametrize("rows,n,cid", [(1300, 2796, 2), (1500, 1060, 2), (40, 20004, 2), (3, 70004, 2), (1300, 1096, 5),
                                         (2, 33000 + 8, 5), (1400, 2052, 4), (5, 9000 + 4, 4)])
def test_rows_of_whole_lines_plus_a_remainder(hs, oracle, rows, n, cid):
    """Row pitch a multiple of 16 bytes but not of 128: a chunk travels as one box of the row's whole 128-byte lines,
    the remainder of the row by plain loads and stores; both kernels; neighbouring rows must stay untouched."""
    w = workloads.make(cid, rows=rows, n=n, seed=rows * 7 + n)
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        if cid == 4:
            run_linear(hs, oracle, w.tensors, path=path, signed=True, what=f"lines+rest {rows}x{n}/{path}")
        else:
            run_log(hs, oracle, w.tensors, path=path, what=f"lines+rest {rows}x{n}/{path}")


def test_tickets_forced_on_few_rows(hs, oracle):
    hs.tune("ROW_TICKETS", 1)
    try:
        for rows, n in ((5, 4100), (300, 515), (2400, 2048)):
            w = workloads.make(2, rows=rows, n=n, seed=rows)
            run_log(hs, oracle, w.tensors, path=hs.PATH_BATCHED, what=f"forced tickets {rows}x{n}")
    finally:
        hs.tune("ROW_TICKETS", -1)


@pytest.mark.parametrize("n", [7, 520, 4099])
def test_odd_shapes_signed_linear(hs, oracle, n):
    w = workloads.make(4, rows=5, n=n, seed=n)
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        run_linear(hs, oracle, w.tensors, path=path, signed=True, what=f"signed 5x{n}/{path}")


@pytest.mark.parametrize("rows,n,cid", [(1800, 1056, 2), (1800, 544, 2), (2, 5 * 512 + 96, 2), (1900, 1088, 5), (3, 7 * 512 + 64, 5)])
def test_rows_on_128_byte_lines_with_partial_last_chunk(hs, oracle, rows, n, cid):
    """Rows that start on 128-byte lines move as single contiguous boxes even when n is not a multiple of
    the chunk; the partial last chunk of every row must not spill into the next row (canaries around the
    output, exact parity inside)."""
    w = workloads.make(cid, rows=rows, n=n)
    t = w.tensors
    la, lb, lx0 = to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"])
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    tol = tol_positive(storage_f64(t["log_a"]), ref)
    if cid == 5:
        tol = tol + 1e-2 * np.abs(ref)
    pad = 4096
    buf = torch.zeros(rows * n + 2 * pad, dtype=la.dtype, device="cuda")
    buf[:pad] = 12345.0
    buf[-pad:] = 12345.0
    out = buf[pad:pad + rows * n].view(rows, n)
    ws = hs.new_workspace(rows, n, "cuda")
    hs.scan_log(la, lb, lx0, log_x=out, workspace=ws)
    hs.check(ws)
    assert_log_close(to_f64(out), ref, tol, f"{rows}x{n}")
    assert (buf[:pad] == 12345.0).all() and (buf[-pad:] == 12345.0).all()


def test_unaligned_base_pointer(hs, oracle):
    w = workloads.make(2, rows=9, n=1000)
    t = w.tensors
    rows, n = 9, 1000
    def shifted(arr):  # base pointer 4 bytes past a 16-byte boundary
        buf = torch.empty(arr.size + 1, dtype=torch.float32, device="cuda")
        v = buf[1:].view(arr.shape)
        v.copy_(torch.from_numpy(arr))
        return v
    la, lb = shifted(t["log_a"]), shifted(t["log_b"])
    out = hs.scan_log(la, lb, to_dev(t["log_x0"]))
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    assert_log_close(to_f64(out), ref, tol_positive(t["log_a"].astype(np.float64), ref), "unaligned base")


# ------------------------------------------------------------------------------------------ degenerate inputs
@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_zeros_resets_and_wide_range(hs, oracle, path):
    """log 0 = -inf inputs, a_t = 0 (state reset), x0 = 0, and runs whose terms span hundreds of
    orders of magnitude (the kernel's tracked form) all reproduce the oracle."""
    rng = np.random.default_rng(11)
    rows, n = 6, 3000
    la = -rng.uniform(0, 0.3, (rows, n)).astype(np.float32)
    lb = rng.normal(size=(rows, n)).astype(np.float32)
    lx0 = rng.normal(size=rows).astype(np.float32)
    lb[0, :] = -np.inf                                  # b == 0 everywhere: log x = log x0 + a*
    lx0[1] = -np.inf                                    # x0 == 0
    lb[1, :700] = -np.inf                               # ... and nothing added for 700 steps: x == 0 exactly
    la[2, [5, 600, 601, 2999]] = -np.inf                # a_t == 0: the state resets to b_t
    lb[3, ::7] = -np.inf                                # sparse zeros
    lb[4, :] = rng.uniform(-300, 300, n).astype(np.float32)   # wide dynamic range inside every run
    la[5, :] = -rng.uniform(5, 30, n).astype(np.float32)      # violent decay: a* ~ -50000
    lx0[5] = 50.0
    t = dict(log_a=la, log_b=lb, log_x0=lx0)
    hs.set_path(getattr(hs, "PATH_" + path.upper()))
    out = hs.scan_log(to_dev(la), to_dev(lb), to_dev(lx0))
    got = to_f64(out)
    ref, _ = oracle.scan_log(la, lb, lx0)
    assert_log_close(got, ref, tol_positive(la.astype(np.float64), ref), f"degenerate/{path}")
    assert np.isneginf(got[1, :700]).all()


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_linear_products_that_leave_fp32_inside_a_run(hs, oracle, path):
    """scan_linear with stretches of tiny and of huge |a_t|: the product of a lane's 16 factors leaves fp32's range
    (below 2^-240 or above 2^240) although every x_t stays representable.  The look-back kernel hands exp(A_t / 2)
    from its first phase to its second and must fall back to the tracked form on such chunks; the row-batched kernel
    keeps A_t itself.  Tiny stretches forget the past (x_t ~ b_t); huge factors are followed by tiny ones."""
    rng = np.random.default_rng(21)
    rows, n = 3, 7168 * 3 + 100
    a = rng.uniform(0.5, 1.0, (rows, n)).astype(np.float32) * rng.choice([-1, 1], (rows, n)).astype(np.float32)
    b = rng.normal(size=(rows, n)).astype(np.float32)
    x0 = rng.normal(size=rows).astype(np.float32)
    a[0, 1000:1400] = rng.choice([-1, 1], 400).astype(np.float32) * np.float32(3e-6)     # 2^-18 each: 2^-290 per run
    a[1, 5000:9000] = rng.choice([-1, 1], 4000).astype(np.float32) * np.float32(1e-7)
    a[2, 300:340:2] = np.float32(2e5)                                                    # up ...
    a[2, 301:341:2] = np.float32(-5e-6)                                                  # ... and down again, pairwise
    a[2, 12000:12020] = np.float32(4e4)                                                  # 20 factors of 2^15: 2^300,
    b[2, 12000:12020] = 0.0
    a[2, 12020:12040] = np.float32(2.5e-5)                                               # taken back by 20 of 2^-15
    b[2, 12020:12040] = 0.0
    b[2, 10000:12000] = 0.0
    a[2, 10000:12000] = np.float32(0.93)                    # x ~ 1e-63 when the climb begins (below fp32, not below the carry)
    hs.set_path(getattr(hs, "PATH_" + path.upper()))
    ws = hs.new_workspace(rows, n, "cuda")
    x = hs.scan_linear(to_dev(a), to_dev(b), to_dev(x0), workspace=ws)
    hs.check(ws)
    ref = oracle.scan_linear(a, b, x0)
    got = to_f64(x)
    assert np.abs(ref).max() < 1e38 and np.isfinite(got).all()
    assert np.abs(ref[2, 12019]) > 1e20                     # the climb really happened
    assert_signed_close(got, ref, f"linear wide range/{path}")
    np.testing.assert_allclose(got[2, 12010:12020], ref[2, 12010:12020], rtol=1e-3)
    # where the past is forgotten the result is b_t to fp32 accuracy, whatever the scale of the row
    np.testing.assert_allclose(got[0, 1001:1400], ref[0, 1001:1400], rtol=2e-5, atol=1e-6)
    np.testing.assert_allclose(got[1, 5001:9000], ref[1, 5001:9000], rtol=2e-5, atol=1e-6)


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_linear_zeros_and_cancellation(hs, oracle, path):
    rng = np.random.default_rng(12)
    rows, n = 4, 2500
    a = rng.uniform(0.5, 1.0, (rows, n)).astype(np.float32) * rng.choice([-1, 1], (rows, n)).astype(np.float32)
    b = rng.normal(size=(rows, n)).astype(np.float32)
    x0 = rng.normal(size=rows).astype(np.float32)
    a[0, [0, 17, 1000]] = 0.0
    b[1, :] = 0.0
    x0[2] = 0.0
    b[2, :40] = 0.0
    a[3, :] = -1.0
    b[3, :] = 0.0                                      # x_t = (-1)^t x0
    hs.set_path(getattr(hs, "PATH_" + path.upper()))
    x = hs.scan_linear(to_dev(a), to_dev(b), to_dev(x0))
    ref = oracle.scan_linear(a, b, x0)
    got = to_f64(x)
    assert_signed_close(got, ref, f"linear degenerate/{path}")
    assert (got[2, :40] == 0).all()
    np.testing.assert_allclose(got[3], ref[3], rtol=1e-5)


def test_nan_and_inf_stay_in_their_row(hs, oracle):
    w = workloads.make(2, rows=8, n=2048)
    t = {k: v.copy() for k, v in w.tensors.items()}
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    t["log_b"][3, 1000] = np.nan
    t["log_a"][5, 77] = np.inf
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        hs.set_path(path)
        got = to_f64(hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"])))
        tol = tol_positive(w.tensors["log_a"].astype(np.float64), ref)
        for r in (0, 1, 2, 4, 6, 7):
            assert_log_close(got[r:r + 1], ref[r:r + 1], tol[r:r + 1], f"row {r}")
        assert_log_close(got[3:4, :1000], ref[3:4, :1000], tol[3:4, :1000], "before the NaN")


def test_in_place_and_guard_bands(hs, oracle):
    """The output may alias an input; nothing outside [rows, n] is written (canaries on both sides)."""
    w = workloads.make(2, rows=37, n=1540)
    t = w.tensors
    rows, n = 37, 1540
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    tol = tol_positive(t["log_a"].astype(np.float64), ref)
    pad = 1024
    for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
        hs.set_path(path)
        buf = torch.full((rows * n + 2 * pad,), float("nan"), device="cuda")
        canary = torch.tensor(0x7FC0DEAD, dtype=torch.int32, device="cuda")
        buf.view(torch.int32)[:pad] = canary
        buf.view(torch.int32)[-pad:] = canary
        out = buf[pad:pad + rows * n].view(rows, n)
        out.copy_(torch.from_numpy(t["log_b"]))          # in situ: log_b is overwritten by log x
        hs.scan_log(to_dev(t["log_a"]), out, to_dev(t["log_x0"]), log_x=out)
        assert_log_close(to_f64(out), ref, tol, "in place")
        assert (buf.view(torch.int32)[:pad] == canary).all() and (buf.view(torch.int32)[-pad:] == canary).all()


def test_split_invariance_on_gpu(hs):
    """[0,n) in one call equals [0,k) then [k,n) restarted from x_k, at chunk and tile borders +-1."""
    w = workloads.make(2, rows=3, n=9000)
    la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
    whole = hs.scan_log(la, lb, lx0)
    for k in (511, 512, 513, 4095, 4096, 4097):
        head = hs.scan_log(la[:, :k].contiguous(), lb[:, :k].contiguous(), lx0)
        tail = hs.scan_log(la[:, k:].contiguous(), lb[:, k:].contiguous(), head[:, -1].contiguous())
        got = torch.cat([head, tail], dim=1)
        assert (got - whole).abs().max().item() < 2e-5


def test_empty_and_invalid_arguments(hs):
    z = torch.empty((0, 16), device="cuda")
    assert hs.scan_log(z, z, torch.empty(0, device="cuda")).shape == (0, 16)
    L = hs.lib()
    a = torch.zeros((2, 8), device="cuda")
    x0 = torch.zeros(2, device="cuda")
    ws = hs.new_workspace(2, 8, "cuda")
    p = lambda t: t.data_ptr()
    assert L.heinsen_scan_log(p(a), p(a), p(x0), p(a), None, None, None, None, 0, 8, 0, 0, p(ws), ws.numel(), None) == 0
    assert L.heinsen_scan_log(None, p(a), p(x0), p(a), None, None, None, None, 2, 8, 0, 0, p(ws), ws.numel(), None) == 1
    assert L.heinsen_scan_log(p(a), p(a), p(x0), p(a), None, None, None, None, -1, 8, 0, 0, p(ws), ws.numel(), None) == 1
    assert L.heinsen_scan_log(p(a), p(a), p(x0), p(a), None, None, None, None, 2, 8, 1, 0, p(ws), ws.numel(), None) == 1
    assert L.heinsen_scan_log(p(a), p(a), p(x0), p(a), None, None, None, None, 2, 8, 0, 0, p(ws), 16, None) == 3
    assert L.heinsen_scan_log(p(a), p(a), p(x0), p(a), p(ws), None, None, None, 2, 8, 0, 0, p(ws), ws.numel(), None) == 1
    assert L.heinsen_scan_linear(p(a), p(a), p(x0), p(a), 2, 8, 1, p(ws), ws.numel(), None) == 1
    torch.cuda.synchronize()


def test_lookback_wait_is_bounded_and_reported(hs):
    """A tile that never publishes makes its successors give up after the poll limit: the call
    reports HS_ERR_LOOKBACK_TIMEOUT, nothing hangs, and the next call works."""
    w = workloads.make(2, rows=1, n=1 << 18)
    la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
    hs.set_path(hs.PATH_LOOKBACK)
    ws = hs.new_workspace(1, 1 << 18, "cuda")
    hs.debug_config(lookback_spin_limit=2000, mute_tile=3)
    hs.scan_log(la, lb, lx0, workspace=ws)
    with pytest.raises(hs.HeinsenScanError) as ei:
        hs.check(ws)
    assert ei.value.status == 5
    hs.debug_config(0, -1)
    good = hs.scan_log(la, lb, lx0, workspace=ws)
    hs.check(ws)
    assert torch.isfinite(good).all()


def test_host_buffer_entry_point(hs, oracle):
    w = workloads.make(2, rows=300, n=2048)
    t = w.tensors
    la, lb, lx0 = (torch.from_numpy(t[k]).pin_memory() for k in ("log_a", "log_b", "log_x0"))
    out = torch.empty_like(la).pin_memory()
    scratch = torch.empty(hs.host_scratch_bytes(300, 2048, torch.float32, torch.float32, False), dtype=torch.uint8,
                          device="cuda")
    hs.scan_log_host(la, lb, lx0, out, scratch)
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    assert_log_close(out.double().numpy(), ref, tol_positive(t["log_a"].astype(np.float64), ref), "host entry")


def test_host_buffer_entry_points_signed_and_linear(hs, oracle):
    """Host buffers with sign tensors (log domain) and the linear entry point, more rows than row blocks."""
    rows, n = 37, 1500
    t = workloads.make(4, rows=rows, n=n, seed=9).tensors
    a, b, x0 = (torch.from_numpy(t[k]).pin_memory() for k in ("a", "b", "x0"))
    x = torch.empty_like(a).pin_memory()
    scratch = torch.empty(hs.host_scratch_bytes(rows, n, torch.float32, torch.float32, True), dtype=torch.uint8, device="cuda")
    hs.scan_linear_host(a, b, x0, x, scratch)
    ref = oracle.scan_linear(t["a"], t["b"], t["x0"])
    assert_signed_close(x.double().numpy(), ref, "host linear")
    # the same recurrence handed over as logarithms of magnitudes and sign bytes
    with np.errstate(divide="ignore"):
        la, lb, lx0 = (torch.from_numpy(np.log(np.abs(t[k])).astype(np.float32)).pin_memory() for k in ("a", "b", "x0"))
    sa, sb, sx0 = (torch.from_numpy(np.signbit(t[k]).astype(np.uint8)).pin_memory() for k in ("a", "b", "x0"))
    lx = torch.empty_like(la).pin_memory()
    sx = torch.empty((rows, n), dtype=torch.uint8).pin_memory()
    hs.scan_log_host(la, lb, lx0, lx, scratch, sign_a=sa, sign_b=sb, sign_x0=sx0, sign_x=sx)
    got = np.exp(lx.double().numpy()) * np.where(sx.numpy() == 1, -1.0, 1.0)
    ref_log, ref_sign = oracle.scan_log(la.numpy(), lb.numpy(), lx0.numpy(), sa.numpy(), sb.numpy(), sx0.numpy())
    assert_signed_close(got, np.exp(ref_log) * np.where(ref_sign == 1, -1.0, 1.0), "host log with signs")


@pytest.mark.parametrize("rows,n,kind", [
    (3, 7168 * 40 + 5, "log"),      # 41 tiles per row: rows begin in the middle of the carry server's 32-tile batches
    (70, 7168 * 2 + 1, "log"),      # 3 tiles per row: ten rows begin inside every batch
    (1, 7168 * 32, "log"),          # exactly one batch
    (1, 7168 * 33, "log"),          # one batch and one tile
    (1, 7168 * 1030 + 17, "log"),   # more batches than the server's hand-over ring has slots, twice over
    (33, 7168 * 31 + 100, "linear"),  # signed values cross tiles, batches and rows
    (2, 7168 * 100 + 3, "bf16"),
])
def test_lookback_carry_server_batches(hs, oracle, rows, n, kind):
    """The value of x entering each tile of the single-pass kernel comes from the grid's last CTA, whose warps scan
    the tiles' aggregates 32 tiles at a time and hand the running value from batch to batch; rows begin anywhere
    inside a batch.  Every element against the oracle."""
    if kind == "linear":
        w = workloads.make(4, rows=rows, n=n)
        run_linear(hs, oracle, w.tensors, path=hs.PATH_LOOKBACK, signed=True, what=f"{rows} x {n} linear")
    else:
        w = workloads.make(5 if kind == "bf16" else 3, rows=rows, n=n)
        run_log(hs, oracle, w.tensors, path=hs.PATH_LOOKBACK, what=f"{rows} x {n} {kind}")


@pytest.mark.parametrize("path", ["batched", "lookback"])
def test_workspace_needs_no_initialisation(hs, oracle, path):
    """The workspace may hold anything: random bytes, or what a call on another problem left there.  Every word a
    kernel reads from it (row tickets, hand-over words, the tiles' aggregates and entering values) counts only if it
    carries this call's id."""
    hs.set_path(getattr(hs, "PATH_" + path.upper()))
    shapes = [(3, 7168 * 9 + 100), (2, 7168 * 40)] if path == "lookback" else [(2500, 2048), (9000, 600)]
    nbytes = max(hs.workspace_bytes(r, n) for r, n in shapes)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda")
    g.manual_seed(1234)
    for fill in ("random", "ones", "previous call", "previous call"):
        if fill == "random":
            ws.copy_(torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device="cuda", generator=g))
        elif fill == "ones":
            ws.fill_(0xFF)
        for rows, n in shapes:  # (the second shape runs on what the first one left, and the next round on both)
            w = workloads.make(3 if path == "lookback" else 2, rows=rows, n=n, seed=rows)
            t = w.tensors
            out = hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]), workspace=ws)
            hs.check(ws)
            ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
            assert_log_close(to_f64(out), ref, tol_positive(t["log_a"].astype(np.float64), ref), f"{fill}, {rows} x {n}")


def test_lookback_several_rows_several_groups(hs, oracle):
    """Single-pass path with a few rows, each several rounds of tiles long, plus a ragged last tile: the carry
    crosses tiles, batches of tiles and the row starts inside a launch."""
    rows, n = 3, 2_650_112 + 40
    w = workloads.make(3, rows=rows, n=n)
    t = w.tensors
    hs.set_path(hs.PATH_LOOKBACK)
    ws = hs.new_workspace(rows, n, "cuda")
    out = hs.scan_log(to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"]), workspace=ws)
    hs.check(ws)
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    assert_log_close(to_f64(out), ref, tol_positive(t["log_a"].astype(np.float64), ref), "3 rows x 2.65M")


@pytest.mark.parametrize("path", ["batched", "lookback"])
@pytest.mark.parametrize("rows,n,offset", [(40, 3000, 0), (37, 3001, 0), (40, 3000, 1), (2000, 100, 0), (1900, 37, 0),
                                            (3, 70004, 0), (2, 70001, 1), (300, 256, 0), (5, 1, 0)])
def test_complex_logarithm_interface(hs, oracle, path, rows, n, offset):
    """Negative a, b, x0 as complex logarithms (log r + i*pi): the result is real, i.e. its imaginary part is
    0 or pi, and exp of it equals the recurrence in the linear domain.  Shapes: rows of whole 16-byte units with
    and without a remainder of the last 128-byte line, an odd number of elements per row and a base that is only
    8-byte aligned (rows TMA cannot address), rows shorter than a chunk (several rows per warp), long rows."""
    w = workloads.make(4, rows=rows, n=n)
    a, b, x0 = (w.tensors[k].astype(np.float64) for k in ("a", "b", "x0"))
    with np.errstate(divide="ignore"):
        la, lb, lx0 = (np.log(v.astype(np.complex128)).astype(np.complex64) for v in (a, b, x0))
    la.imag[:, ::3] += np.float32(2 * np.pi)         # any odd/even multiple of pi is the same sign
    lb.imag[:, 1::5] -= np.float32(2 * np.pi)
    hs.set_path(getattr(hs, "PATH_" + path.upper()))

    def place(v):   # at `offset` elements into a larger buffer: offset 1 leaves the base 8-byte aligned only
        buf = torch.empty(v.size + 2, dtype=torch.complex64, device="cuda")
        view = buf[offset:offset + v.size].view(v.shape)
        view.copy_(torch.from_numpy(v))
        return view

    d_la, d_lb, d_lx0 = place(la), place(lb), torch.from_numpy(lx0).cuda()
    out_buf = torch.full((rows * n + 2,), float("nan"), dtype=torch.complex64, device="cuda")
    out = out_buf[offset:offset + rows * n].view(rows, n)
    hs.scan_log_complex(d_la, d_lb, d_lx0, log_x=out)
    torch.cuda.synchronize()
    z = out.cpu().numpy()
    edge = out_buf.cpu().numpy()
    assert np.isnan(edge[:offset].real).all() and np.isnan(edge[offset + rows * n:].real).all(), "wrote outside the output"
    assert np.isin(np.round(z.imag / np.pi), (0, 1)).all() and np.allclose(z.imag, np.round(z.imag / np.pi) * np.pi, atol=1e-6)
    got = np.exp(z.real.astype(np.float64)) * np.where(np.round(z.imag / np.pi) == 1, -1.0, 1.0)
    ref = oracle.scan_linear(w.tensors["a"], w.tensors["b"], w.tensors["x0"])
    assert_signed_close(got, ref, f"complex interface/{path} {rows}x{n}+{offset}")
    # the same values through the sign + magnitude entry point: same kernels apart from where the sign bit comes from
    mag = lambda v: torch.from_numpy(np.ascontiguousarray(v.real)).cuda()
    sgn = lambda v: torch.from_numpy((np.round(v.imag / np.pi).astype(np.int64) & 1).astype(np.uint8)).cuda()
    lx2, sx2 = hs.scan_log(mag(la), mag(lb), mag(lx0), sign_a=sgn(la), sign_b=sgn(lb), sign_x0=sgn(lx0))
    torch.cuda.synchronize()
    got2 = np.exp(to_f64(lx2)) * np.where(sx2.cpu().numpy() == 1, -1.0, 1.0)
    assert_signed_close(got2, ref, "sign + magnitude entry point on the same values")
    assert np.abs(got - got2).max() <= 2e-3 * np.abs(ref).max()   # (near a cancellation log|x| itself is ill-conditioned)


def test_short_forms_of_the_two_calls(hs, oracle):
    """scan_linear(a, b, x0, x, rows, n) and scan_log(..., rows, n): fp32, default stream, library scratch."""
    L = hs.lib()
    w = workloads.make(4, rows=1300, n=1024)
    a, b, x0 = (to_dev(w.tensors[k]) for k in ("a", "b", "x0"))
    x = torch.empty_like(a)
    torch.cuda.synchronize()
    assert L.scan_linear(a.data_ptr(), b.data_ptr(), x0.data_ptr(), x.data_ptr(), 1300, 1024) == 0
    hs.check_static("cuda")
    assert_signed_close(to_f64(x), oracle.scan_linear(w.tensors["a"], w.tensors["b"], w.tensors["x0"]), "scan_linear short form")
    w = workloads.make(3, rows=1, n=1 << 20)
    la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
    out = torch.empty_like(la)
    torch.cuda.synchronize()
    assert L.scan_log(la.data_ptr(), lb.data_ptr(), lx0.data_ptr(), out.data_ptr(), None, None, None, None, 1, 1 << 20) == 0
    hs.check_static("cuda")
    ref, _ = oracle.scan_log(w.tensors["log_a"], w.tensors["log_b"], w.tensors["log_x0"])
    assert_log_close(to_f64(out), ref, tol_positive(w.tensors["log_a"].astype(np.float64), ref), "scan_log short form")


@pytest.mark.parametrize("seed", range(10))
def test_random_shapes_all_modes(hs, oracle, seed):
    """Seeded random shapes (short and long rows, few and many, aligned and not) through every mode and both kernels."""
    rng = np.random.default_rng(1000 + seed)
    for _ in range(5):
        n = int(rng.choice([rng.integers(1, 40), rng.integers(40, 700), rng.integers(700, 6000), rng.integers(6000, 40000)]))
        if rng.random() < 0.5:
            n = max(4, n // 4 * 4)  # a pitch that TMA can address
        rows = int(rng.choice([rng.integers(1, 8), rng.integers(8, 400), rng.integers(400, 6000)]))
        rows = max(1, min(rows, 3_000_000 // n))
        cid = int(rng.choice([2, 4, 5]))
        w = workloads.make(cid, rows=rows, n=n, seed=seed)
        for path in (hs.PATH_BATCHED, hs.PATH_LOOKBACK):
            what = f"random cfg{cid} {rows}x{n}/{path}"
            if cid == 4:
                run_linear(hs, oracle, w.tensors, path=path, signed=True, what=what)
            else:
                run_log(hs, oracle, w.tensors, path=path, what=what)


def test_two_streams_with_their_own_workspaces(hs):
    """Calls on two streams may overlap on the GPU; each has its own workspace (ticket word, descriptors)."""
    shapes = [(20000, 2048, 2), (3, 300000, 2), (9000, 4096, 2), (1, 1 << 20, 2)]
    data = []
    for rows, n, cid in shapes:
        t = workloads.make(cid, rows=rows, n=n, seed=rows).tensors
        la, lb, lx0 = to_dev(t["log_a"]), to_dev(t["log_b"]), to_dev(t["log_x0"])
        ws = hs.new_workspace(rows, n, "cuda")
        ref = hs.scan_log(la, lb, lx0, workspace=ws)
        hs.check(ws)
        data.append((la, lb, lx0, ref.clone()))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs, wss = [], []
    for rep in range(3):
        for k, (la, lb, lx0, ref) in enumerate(data):
            with torch.cuda.stream(streams[k % 2]):
                ws = hs.new_workspace(la.shape[0], la.shape[1], "cuda")
                outs.append((hs.scan_log(la, lb, lx0, workspace=ws), ref))
                wss.append(ws)
    torch.cuda.synchronize()
    for ws in wss:
        hs.check(ws)
    for out, ref in outs:
        assert torch.equal(out, ref)


def test_repeatability(hs):
    w = workloads.make(3, rows=1, n=1 << 21)
    la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
    first = hs.scan_log(la, lb, lx0)
    for _ in range(5):
        again = hs.scan_log(la, lb, lx0)
        assert (again - first).abs().max().item() < 1e-5


def test_lookback_abort_with_several_tiles_per_cta_returns_promptly(hs):
    """The same muted tile on a row long enough that every CTA owns several tiles: once the compute warps of a
    CTA have given up, its publisher warp must leave too instead of polling its barrier to the limit.  The call
    has to come back within a fraction of a second and report the time-out."""
    import time
    n = 1 << 22                                     # 586 tiles on 148 CTAs: about four tiles per CTA
    w = workloads.make(2, rows=1, n=n)
    la, lb, lx0 = (to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0"))
    hs.set_path(hs.PATH_LOOKBACK)
    ws = hs.new_workspace(1, n, "cuda")
    hs.debug_config(lookback_spin_limit=2000, mute_tile=3)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    hs.scan_log(la, lb, lx0, workspace=ws)
    with pytest.raises(hs.HeinsenScanError) as ei:
        hs.check(ws)
    elapsed = time.perf_counter() - t0
    assert ei.value.status == 5
    assert elapsed < 2.0, f"aborting launch took {elapsed:.2f} s"
    hs.debug_config(0, -1)
    good = hs.scan_log(la, lb, lx0, workspace=ws)
    hs.check(ws)
    assert torch.isfinite(good).all()


def test_lookback_protocol_stress_smallest_tiles(hs, oracle):
    """Thousands of tiles of the smallest size (8 compute warps) exercise the descriptor protocol a hundred
    times over; every repetition must match the oracle (every wait stays bounded)."""
    n = (1 << 23) + 4096 + 12
    w = workloads.make(3, rows=1, n=n)
    t = w.tensors
    la, lb, lx0 = (to_dev(t[k]) for k in ("log_a", "log_b", "log_x0"))
    ref, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    tol = tol_positive(t["log_a"].astype(np.float64), ref)
    ref_dev = torch.from_numpy(ref).cuda()
    tol_dev = torch.from_numpy(tol).cuda()
    hs.set_path(hs.PATH_LOOKBACK)
    hs.tune("LB_WARPS", 8)
    try:
        ws = hs.new_workspace(1, n, "cuda")
        out = torch.empty_like(la)
        for rep in range(100):
            out.fill_(float("nan"))
            hs.scan_log(la, lb, lx0, log_x=out, workspace=ws)
            hs.check(ws)
            worst = ((out.double() - ref_dev).abs() / tol_dev).max().item()
            assert worst <= 1.0, f"repetition {rep}: {worst:.3g} of the tolerance"
            # the carry between the tiles is composed in a fixed order (batches of 32 tiles, one after the other),
            # whatever the order in which the tiles finish: every repetition gives the same bits
            if rep == 0:
                first = out.clone()
            else:
                assert torch.equal(out, first), f"repetition {rep} differs from the first"
    finally:
        hs.tune("LB_WARPS", -1)


@pytest.mark.parametrize("rows,n,kind", [
    (2500, 2048, "log"), (3000, 1536, "log"), (2369, 1024, "log"), (3001, 5000, "log"), (2600, 4090, "log"),
    (2500, 2048, "linear"), (3000, 3001, "linear"), (2500, 4096, "bf16"), (2900, 1500, "bf16"), (2450, 2050, "complex"),
    (7000, 1030, "log"),
])
def test_rows_shared_out_by_chunks(hs, oracle, rows, n, kind):
    """Between one and a few rows per warp slot the batched kernel cuts the rows to measure: every slot takes an equal
    share of the rows' chunks -- the rest of a row, whole rows, the beginning of a row -- and the value of x crosses
    from slot to slot through the workspace.  Forced on (the automatic choice takes it only where whole rows per slot
    would leave slots idle) and compared with the oracle; forced off, the results must be the same bits."""
    hs.set_path(hs.PATH_BATCHED)
    outs = []
    for spans in (1, 0):
        hs.tune("SPANS", spans)
        try:
            if kind == "linear":
                w = workloads.make(4, rows=rows, n=n, seed=rows)
                x = hs.scan_linear(*(to_dev(w.tensors[k]) for k in ("a", "b", "x0")))
                torch.cuda.synchronize()
                if spans:
                    assert_signed_close(to_f64(x), oracle.scan_linear(w.tensors["a"], w.tensors["b"], w.tensors["x0"]), f"spans {rows}x{n}")
                outs.append(x)
            elif kind == "complex":
                w = workloads.make(4, rows=rows, n=n, seed=rows)
                with np.errstate(divide="ignore"):
                    z = [np.log(w.tensors[k].astype(np.complex128)).astype(np.complex64) for k in ("a", "b", "x0")]
                zo = hs.scan_log_complex(*(torch.from_numpy(v).cuda() for v in z))
                torch.cuda.synchronize()
                if spans:
                    zz = zo.cpu().numpy()
                    got = np.exp(zz.real.astype(np.float64)) * np.where(np.round(zz.imag / np.pi) == 1, -1.0, 1.0)
                    assert_signed_close(got, oracle.scan_linear(w.tensors["a"], w.tensors["b"], w.tensors["x0"]), f"spans complex {rows}x{n}")
                outs.append(torch.view_as_real(zo))
            else:
                w = workloads.make(5 if kind == "bf16" else 2, rows=rows, n=n, seed=rows)
                if spans:
                    run_log(hs, oracle, w.tensors, path=hs.PATH_BATCHED, what=f"spans {kind} {rows}x{n}")
                out = hs.scan_log(*(to_dev(w.tensors[k]) for k in ("log_a", "log_b", "log_x0")))
                torch.cuda.synchronize()
                outs.append(out)
        finally:
            hs.tune("SPANS", -1)
    a, b = outs
    same = (a == b) | (torch.isnan(a) & torch.isnan(b))
    assert same.all(), "the same chunks in another order of slots must give the same bits"
