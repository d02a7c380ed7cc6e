"""Writes theorem2_runtime.txt: the paper's Theorem 2 closed forms evaluated with exact rationals.

Columns: learners, lambda, E[T_nonblocking] = 1/(lambda*P), E[T_dpsgd] = (P/lambda) sum_{k=0}^{P-1} C(P-1,k)(-1)^k/(k+1)^2.
"""
import os
from fractions import Fraction
from math import comb


def t_nonblocking(P, lam):
    return Fraction(1) / (lam * P)


def t_dpsgd(P, lam):
    s = Fraction(0)
    for k in range(P):
        s += Fraction(comb(P - 1, k) * (-1) ** k, (k + 1) ** 2)
    return Fraction(P) / lam * s


if __name__ == "__main__":
    here = os.path.dirname(os.path.abspath(__file__))
    with open(os.path.join(here, "theorem2_runtime.txt"), "w") as f:
        f.write("# Theorem 2 (expected run-time per iteration, exponential mini-batch times), exact rationals -> 17 digits\n")
        f.write("# learners lambda E_T_nonblocking E_T_dpsgd\n")
        for P in (4, 8, 10, 16, 32):
            for lam in (Fraction(1), Fraction(2)):
                f.write("%d %s %.17g %.17g\n" % (P, float(lam), float(t_nonblocking(P, lam)), float(t_dpsgd(P, lam))))
