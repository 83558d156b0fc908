"""Writes eq3_closed_form.txt: the closed forms of the hard-concrete gate
(Eq. 3 with temperature, and the same derivation for the upper clamp) at the
constants every workload uses, evaluated with the scalar math library only."""
import math
import os

BETA, GAMMA, ZETA = 2.0 / 3.0, -0.1, 1.1

if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "eq3_closed_form.txt")
    with open(path, "w") as f:
        f.write("# Closed forms of the hard-concrete gate at beta=2/3, gamma=-0.1, zeta=1.1.\n")
        f.write("# col 1: alpha; col 2: P(z>0) = sigmoid(alpha - beta*log(-gamma/zeta))  (Eq. 3 with temperature beta);\n")
        f.write("# col 3: P(z=1) = sigmoid(alpha - beta*log((1-gamma)/(zeta-1)))  (same derivation, upper clamp).\n")
        f.write("# Written by tests/golden/make_eq3_table.py with the scalar math library only.\n")
        for a in [-3.0, -1.0, 0.0, 0.5, 1.0, 2.0, 3.0]:
            p0 = 1 / (1 + math.exp(-(a - BETA * math.log(-GAMMA / ZETA))))
            p1 = 1 / (1 + math.exp(-(a - BETA * math.log((1 - GAMMA) / (ZETA - 1)))))
            f.write(f"{a:.1f} {p0:.6f} {p1:.6f}\n")
