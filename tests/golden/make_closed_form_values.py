"""Writes closed_form_values.txt from exact rational arithmetic (python fractions only).

The paper prints no worked numeric example for the layer; these are the values its closed
forms (Eq. N(t), Eq. T_thres with tau = 0.95) take at the benchmark shapes, evaluated
without floating point so that they can pin the oracle's implementation of the formulas.
Run:  python tests/golden/make_closed_form_values.py
"""
import os
from fractions import Fraction

ROWS_N = [(8, 2, 16), (60, 4, 16), (64, 8, 8), (256, 8, 16), (256, 8, 96)]
ROWS_T = [(8, 2), (60, 4), (64, 8), (256, 8)]


def main():
    lines = ["# kind E K t_or_tau value   (Eq. N(t) / Eq. T_thres, exact rational arithmetic)"]
    for E, K, t in ROWS_N:
        n = E * (1 - Fraction(E - K, E) ** t)
        lines.append("N %d %d %d %.9f" % (E, K, t, float(n)))
    for E, K in ROWS_T:
        t = 1
        while 1 - Fraction(E - K, E) ** t < Fraction(95, 100):
            t += 1
        lines.append("T_thres %d %d 0.95 %d" % (E, K, t))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_form_values.txt")
    with open(path, "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
