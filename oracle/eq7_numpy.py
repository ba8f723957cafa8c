"""The paper's two-prefix-sum expression written out with numpy's library scans,
in float64 / complex128 -- TEST INFRASTRUCTURE ONLY.

This is not the oracle (the oracle is the sequential recurrence in
``heinsen_oracle.c``).  It restates the *method* literally, one library call
per operator of Eq. 2 and Eq. 7-8, so that the tests can check that the
recurrence and the expression the CUDA kernels fuse are the same function
(Proof section, Eq. 4-6).  Single sequence, no batching, no blocking.
"""
from __future__ import annotations

import numpy as np


def eq7_positive(a, b, x0):
    """Eq. 7 for a_t, b_t, x_0 > 0:  x = exp(a* + tail(LCSE(cat(log x0, log b - a*))))."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    with np.errstate(divide="ignore"):
        a_star = np.cumsum(np.log(a))                            # Eq. 2, first prefix sum
        z = np.concatenate(([np.log(np.float64(x0))], np.log(b) - a_star))  # cat(.)
    lcse = np.logaddexp.accumulate(z)                            # Eq. 8, LogCumSumExp
    return np.exp(a_star + lcse[1:])                             # tail(.), then Eq. 3


def eq3_direct(a, b, x0):
    """Eq. 1-3 without the stabilisation: x = exp(a* + log(x0 + b*)), b* = cumsum exp(log b - a*)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    a_star = np.cumsum(np.log(a))
    b_star = np.cumsum(np.exp(np.log(b) - a_star))
    return np.exp(a_star + np.log(x0 + b_star))


def eq7_complex(a, b, x0):
    """Eq. 7 with the interim logarithms in C (Summary, last paragraph).

    Any sign of a_t, b_t, x_0.  Returns the complex result; its imaginary part
    must vanish up to rounding because x_t is real.
    """
    a = np.asarray(a, dtype=np.complex128)
    b = np.asarray(b, dtype=np.complex128)
    with np.errstate(divide="ignore"):
        a_star = np.cumsum(np.log(a))
        z = np.concatenate(([np.log(np.complex128(x0))], np.log(b) - a_star))
    ref = np.max(z.real[np.isfinite(z.real)]) if np.any(np.isfinite(z.real)) else 0.0
    with np.errstate(divide="ignore"):
        lcse = np.log(np.cumsum(np.exp(z - ref))) + ref          # log-sum-exp trick, one reference
    return np.exp(a_star + lcse[1:])
