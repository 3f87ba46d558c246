"""Writes ns_scalar_iterates.txt: the first five iterates of the scalar quintic
p(x) = a x + b x^3 + c x^5 with the coefficients printed in the paper
(Section 2, "Muon": a, b, c = 3.4445, -4.7750, 2.0315), from several starting
points, in exact rational arithmetic (fractions.Fraction), rounded to 15
significant digits only when printed.  Uses nothing but the Python standard
library, so the values do not depend on the oracle or on any GPU code.

    python tests/golden/make_ns_scalar_iterates.py > tests/golden/ns_scalar_iterates.txt
"""
from fractions import Fraction

A, B, C = Fraction("3.4445"), Fraction("-4.7750"), Fraction("2.0315")
STARTS = ["1", "0.5", "0.1", "0.01", "0.001"]

print("# x0  p(x0)  p^2(x0)  p^3(x0)  p^4(x0)  p^5(x0)   (Section 2 'Muon' coefficients; exact rationals, printed to 15 digits)")
for s in STARTS:
    x = Fraction(s)
    row = [s]
    for _ in range(5):
        x = A * x + B * x ** 3 + C * x ** 5
        row.append("%.15e" % float(x))
    print(" ".join(row))
