"""Writes constant_ab_closed_form.txt: x_t = a^t x0 + b (1 - a^t)/(1 - a) for a = 19/20,
b = 1/2, x0 = 1, i.e. x_t = 10 - 9 (19/20)^t, evaluated in exact rational arithmetic and
printed to 20 significant digits.  Uses only the Python standard library (no oracle, no CUDA).

Source of the formula: geometric-series closed form of the recurrence x_t = a x_{t-1} + b
(the paper's Eq. 4 with constant a_t, b_t).  Run:  python tests/golden/make_constant_ab_golden.py
"""
from decimal import Decimal, getcontext
from fractions import Fraction
import os

getcontext().prec = 40
a, b, x0 = Fraction(19, 20), Fraction(1, 2), Fraction(1)
ts = [1, 2, 3, 4, 5, 10, 16, 50, 100, 500, 1000, 4096]
here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "constant_ab_closed_form.txt"), "w") as f:
    f.write("# x_t = 10 - 9*(19/20)^t  (closed form of x_t = 0.95 x_{t-1} + 0.5, x_0 = 1; Eq. 4 with constant a, b)\n")
    f.write("# t  x_t (exact rational, rounded to 20 significant digits)\n")
    for t in ts:
        x = a ** t * x0 + b * (1 - a ** t) / (1 - a)
        d = Decimal(x.numerator) / Decimal(x.denominator)
        f.write(f"{t} {d:.20g}\n")
