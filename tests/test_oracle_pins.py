"""Pins for the float64 CPU oracle (no GPU needed).

The oracle is the sequential recurrence x_t = a_t x_{t-1} + b_t.  These tests tie it to
things other than itself: a closed form in exact rational arithmetic (golden file), a
library cumulative sum, a rational brute force of the paper's Eq. 4, the paper's Eq. 1-3 and
Eq. 7-8 restated with numpy's library scans (real and complex-log paths), and invariants
that a dropped term, a wrong sign, an off-by-one index or swapped operands would break.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import eq7_numpy
from paper_2311_06281_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- closed forms
def test_constant_ab_matches_golden_closed_form(oracle):
    # x_t = 10 - 9*0.95^t (golden file, exact rational arithmetic, see its generator script)
    rows = [l.split() for l in open(os.path.join(GOLDEN, "constant_ab_closed_form.txt")) if not l.startswith("#")]
    n = 4096
    a = np.full((1, n), 0.95, dtype=np.float64)
    b = np.full((1, n), 0.5, dtype=np.float64)
    x = oracle.scan_linear(a, b, np.ones(1))[0]
    lx, sx = oracle.scan_log(np.log(a), np.log(b), np.zeros(1))
    for t, v in rows:
        t, v = int(t), float(v)
        assert x[t - 1] == pytest.approx(v, rel=1e-13), t
        assert lx[0, t - 1] == pytest.approx(np.log(v), abs=1e-12), t
    assert not sx.any()


def test_constant_ab_fp32_storage_is_widened_exactly(oracle):
    # With float32 storage the oracle must see the *stored* a = fp32(0.95), not 0.95.
    a32 = np.float32(0.95)
    fa, fb = Fraction(float(a32)), Fraction(1, 2)
    n = 64
    x = oracle.scan_linear(np.full((1, n), a32), np.full((1, n), 0.5, np.float32), np.ones(1, np.float32))[0]
    for t in (1, 2, 17, 64):
        exact = fa ** t + fb * (1 - fa ** t) / (1 - fa)
        assert x[t - 1] == pytest.approx(float(exact), rel=1e-14)
    # and it differs measurably from the 0.95 answer, so a silent re-rounding would be caught
    assert abs(x[63] - (10 - 9 * 0.95 ** 64)) > 1e-8


def test_a_equal_one_is_cumsum(oracle):
    rng = np.random.default_rng(1)
    b = rng.normal(size=(3, 1000))
    x0 = rng.normal(size=3)
    x = oracle.scan_linear(np.ones_like(b), b, x0)
    np.testing.assert_allclose(x, x0[:, None] + np.cumsum(b, axis=1), rtol=0, atol=1e-11)


def test_b_zero_isolates_first_prefix_sum(oracle):
    rng = np.random.default_rng(2)
    la = -rng.uniform(0, 1, size=(2, 300))
    lx0 = rng.normal(size=2)
    lx, _ = oracle.scan_log(la, np.full_like(la, -np.inf), lx0)
    np.testing.assert_allclose(lx, lx0[:, None] + np.cumsum(la, axis=1), rtol=0, atol=1e-11)


def test_a_one_x0_zero_isolates_logcumsumexp(oracle):
    rng = np.random.default_rng(3)
    lb = rng.normal(scale=4.0, size=(2, 500))
    lx, _ = oracle.scan_log(np.zeros_like(lb), lb, np.full(2, -np.inf))
    np.testing.assert_allclose(lx, np.logaddexp.accumulate(lb, axis=1), rtol=0, atol=1e-11)


# --------------------------------------------------------------------------- Eq. 4 brute force
def _eq4_fraction(a, b, x0):
    """x_t = sum_{s=0..t} b_s prod_{r=s+1..t} a_r with b_0 := x_0 (expansion in the Proof section)."""
    n = len(a)
    out = []
    for t in range(1, n + 1):
        tot = Fraction(0)
        for s in range(0, t + 1):
            term = x0 if s == 0 else b[s - 1]
            for r in range(s + 1, t + 1):
                term = term * a[r - 1]
            tot += term
        out.append(tot)
    return out


def _dyadic(rng, size, scale=8):
    return [Fraction(int(v), scale) for v in rng.integers(-3 * scale, 3 * scale + 1, size=size)]


def test_bruteforce_all_sign_patterns_small_n(oracle):
    mags_a = [Fraction(3, 4), Fraction(5, 4), Fraction(1, 2), Fraction(7, 8)]
    mags_b = [Fraction(1, 2), Fraction(3, 2), Fraction(1, 4), Fraction(2)]
    for n in (1, 2, 3, 4):
        for signs in itertools.product((1, -1), repeat=2 * n + 1):
            a = [signs[i] * mags_a[i] for i in range(n)]
            b = [signs[n + i] * mags_b[i] for i in range(n)]
            x0 = signs[2 * n] * Fraction(3, 8)
            ref = np.array([float(v) for v in _eq4_fraction(a, b, x0)])
            af = np.array([[float(v) for v in a]])
            bf = np.array([[float(v) for v in b]])
            x = oracle.scan_linear(af, bf, np.array([float(x0)]))[0]
            np.testing.assert_allclose(x, ref, rtol=1e-14, atol=1e-15)
            lx, sx = oracle.scan_log(np.log(np.abs(af)), np.log(np.abs(bf)), np.log(np.abs([float(x0)])),
                                     (af < 0), (bf < 0), np.array([x0 < 0]))
            xs = np.where(sx[0] == 1, -1.0, 1.0) * np.exp(lx[0])
            np.testing.assert_allclose(xs, ref, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("seed", range(6))
def test_bruteforce_random_up_to_16(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(5, 17))
    a, b = _dyadic(rng, n), _dyadic(rng, n)
    x0 = _dyadic(rng, 1)[0]
    ref = np.array([float(v) for v in _eq4_fraction(a, b, x0)])
    af = np.array([[float(v) for v in a]])
    bf = np.array([[float(v) for v in b]])
    x = oracle.scan_linear(af, bf, np.array([float(x0)]))[0]
    np.testing.assert_allclose(x, ref, rtol=1e-13, atol=1e-13)
    with np.errstate(divide="ignore"):
        lx, sx = oracle.scan_log(np.log(np.abs(af)), np.log(np.abs(bf)), np.log(np.abs([float(x0)])),
                                 (af < 0), (bf < 0), np.array([x0 < 0]))
    xs = np.where(sx[0] == 1, -1.0, 1.0) * np.exp(lx[0])
    np.testing.assert_allclose(xs, ref, rtol=1e-11, atol=1e-11 * max(1.0, np.abs(ref).max()))


# --------------------------------------------------------------------------- the paper's expression
def test_recurrence_equals_eq7_positive(oracle):
    rng = np.random.default_rng(4)
    n = 2000
    a = rng.uniform(0.8, 1.1, n)
    b = rng.uniform(0.0, 2.0, n)
    x0 = 0.7
    x = oracle.scan_linear(a[None], b[None], np.array([x0]))[0]
    np.testing.assert_allclose(eq7_numpy.eq7_positive(a, b, x0), x, rtol=1e-10)
    np.testing.assert_allclose(eq7_numpy.eq3_direct(a, b, x0), x, rtol=1e-10)
    lx, _ = oracle.scan_log(np.log(a)[None], np.log(b)[None], np.log([x0]))
    np.testing.assert_allclose(lx[0], np.log(x), rtol=0, atol=1e-10)


def test_recurrence_equals_eq7_complex_log_path(oracle):
    # negatives: interim logs in C, result real (Summary, last paragraph)
    rng = np.random.default_rng(5)
    n = 400
    a = rng.uniform(0.5, 1.0, n) * rng.choice([-1.0, 1.0], n)
    b = rng.normal(size=n)
    x0 = -0.3
    x = oracle.scan_linear(a[None], b[None], np.array([x0]))[0]
    xc = eq7_numpy.eq7_complex(a, b, x0)
    scale = np.abs(x).max()
    assert np.abs(xc.imag).max() < 1e-9 * scale
    np.testing.assert_allclose(xc.real, x, rtol=0, atol=1e-9 * scale)
    lx, sx = oracle.scan_log(np.log(np.abs(a))[None], np.log(np.abs(b))[None], np.log([abs(x0)]),
                             (a < 0)[None], (b < 0)[None], np.array([1], np.uint8))
    np.testing.assert_allclose(np.where(sx[0] == 1, -1.0, 1.0) * np.exp(lx[0]), x, rtol=0, atol=1e-9 * scale)


# --------------------------------------------------------------------------- invariants
def test_sign_identity_pins_parity_logic(oracle):
    # a -> -a, b_t -> (-1)^t b_t  ==>  x_t -> (-1)^t x_t
    rng = np.random.default_rng(6)
    n = 257
    a = rng.uniform(0.5, 1.2, n)
    b = rng.normal(size=n)
    alt = (-1.0) ** np.arange(1, n + 1)
    x = oracle.scan_linear(a[None], b[None], np.array([0.4]))[0]
    y = oracle.scan_linear((-a)[None], (alt * b)[None], np.array([0.4]))[0]
    np.testing.assert_allclose(y, alt * x, rtol=1e-12, atol=1e-12)
    lx, sx = oracle.scan_log(np.log(a)[None], np.log(np.abs(b))[None], np.log([0.4]),
                             np.ones((1, n), np.uint8), ((alt * b) < 0)[None], None)
    np.testing.assert_allclose(np.where(sx[0] == 1, -1.0, 1.0) * np.exp(lx[0]), alt * x, rtol=1e-10, atol=1e-12)


def test_log_domain_scaling_has_no_hidden_overflow(oracle):
    # (x0, b) -> (c x0, c b) ==> log x -> log x + log c, for c = e^{+-600}
    rng = np.random.default_rng(7)
    la = -rng.uniform(0, 0.3, size=(1, 500))
    lb = rng.normal(size=(1, 500))
    lx0 = np.array([0.2])
    base, _ = oracle.scan_log(la, lb, lx0)
    for c in (600.0, -600.0):
        shifted, _ = oracle.scan_log(la, lb + c, lx0 + c)
        np.testing.assert_allclose(shifted - c, base, rtol=0, atol=1e-9)


def test_split_invariance(oracle):
    # associativity footnote: [0,n) in one call == [0,k) then [k,n) restarted from x_k
    rng = np.random.default_rng(8)
    n, k = 300, 117
    a = rng.uniform(0.5, 1.0, (1, n)) * rng.choice([-1.0, 1.0], (1, n))
    b = rng.normal(size=(1, n))
    x = oracle.scan_linear(a, b, np.array([1.5]))
    head = oracle.scan_linear(a[:, :k], b[:, :k], np.array([1.5]))
    tail = oracle.scan_linear(a[:, k:], b[:, k:], head[:, -1])
    np.testing.assert_array_equal(np.concatenate([head, tail], axis=1), x)


def test_rows_are_independent(oracle):
    w = workloads.make(2, rows=8, n=64)
    t = w.tensors
    full, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    for r in (0, 3, 7):
        one, _ = oracle.scan_log(t["log_a"][r:r + 1], t["log_b"][r:r + 1], t["log_x0"][r:r + 1], nthreads=1)
        np.testing.assert_array_equal(one[0], full[r])


def test_zeros_and_reset(oracle):
    # a_t = 0 resets the state to b_t; b_t = 0 and x0 = 0 contribute nothing (log 0 = -inf is legal)
    a = np.array([[0.5, 0.0, 2.0, 1.0]])
    b = np.array([[1.0, 3.0, 0.0, 0.0]])
    x = oracle.scan_linear(a, b, np.array([0.0]))[0]
    np.testing.assert_array_equal(x, [1.0, 3.0, 6.0, 6.0])
    with np.errstate(divide="ignore"):
        lx, sx = oracle.scan_log(np.log(a), np.log(b), np.array([-np.inf]))
    np.testing.assert_allclose(np.exp(lx[0]), [1.0, 3.0, 6.0, 6.0], rtol=1e-15)
    # exact cancellation: +1 then a = 1, b = -1 -> 0 with sign '+'
    lx, sx = oracle.scan_log(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros(1), None, np.ones((1, 1), np.uint8), None)
    assert lx[0, 0] == -np.inf and sx[0, 0] == 0


def test_eq1_residual_is_nondecreasing_for_positive_b(oracle):
    # Eq. 1: log x_t - a*_t = log(x0 + b*_t), and b*_t is a sum of positive terms
    w = workloads.make(2, rows=4, n=512)
    t = w.tensors
    lx, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    astar = np.cumsum(t["log_a"].astype(np.float64), axis=1)
    resid = lx - astar
    assert (np.diff(resid, axis=1) >= -1e-9).all()
    assert (resid[:, 0] >= t["log_x0"].astype(np.float64) - 1e-12).all()


def test_bf16_storage_is_widened_exactly(oracle):
    w = workloads.make(5, rows=2, n=128)
    t = w.tensors
    assert t["log_a"].dtype == np.uint16
    as_f32 = {k: workloads.bf16_bits_to_f32(v) for k, v in t.items()}
    l16, _ = oracle.scan_log(t["log_a"], t["log_b"], t["log_x0"])
    l32, _ = oracle.scan_log(as_f32["log_a"], as_f32["log_b"], as_f32["log_x0"])
    np.testing.assert_array_equal(l16, l32)
    # round-to-nearest-even on the generator side
    assert workloads.to_bf16_bits(np.array([1.00390625]))[0] == 0x3F80       # tie -> even
    assert workloads.to_bf16_bits(np.array([1.01171875]))[0] == 0x3F82       # tie -> even (up)


def test_workloads_are_seeded_and_prefix_consistent():
    a = workloads.make(2, rows=4, n=2048).tensors
    b = workloads.make(2, rows=4, n=2048).tensors
    c = workloads.make(2, rows=8, n=2048).tensors
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    np.testing.assert_array_equal(a["log_a"], c["log_a"][:4])
    w4 = workloads.make(4, rows=2, n=4096).tensors
    frac_neg = (w4["a"] < 0).mean()
    assert 0.4 < frac_neg < 0.6 and np.abs(w4["a"]).min() >= 0.5
