"""Writes entropy_closed_forms.txt: Shannon entropy (nats, Eq. 1) of softmax rows
that have a closed form, evaluated with 60-digit decimal arithmetic.  Calls neither
the oracle nor the CUDA library.

Row family: m entries equal to c, the other V - m entries equal to 0.
    Z = m e^c + (V - m);   H = ln Z - m c e^c / Z        (c = 0: H = ln V)
The c values are exactly representable in fp32 so the row the tests build is the
row evaluated here.
"""
import os
from decimal import Decimal, getcontext

getcontext().prec = 60
CASES = [
    ("uniform", 1024, 0, "0"), ("uniform", 126464, 0, "0"), ("uniform", 152064, 0, "0"),
    ("spike", 1024, 1, "3.5"), ("spike", 126464, 1, "12.25"), ("spike", 126464, 16, "8"),
    ("spike", 152064, 2, "20"), ("spike", 4096, 4000, "-1.5"), ("spike", 32, 1, "0.125"),
]


def entropy(V, m, c):
    c = Decimal(c)
    ec = c.exp()
    Z = m * ec + (V - m)
    return Z.ln() - m * c * ec / Z


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "entropy_closed_forms.txt")
    with open(out, "w") as f:
        f.write("# Closed-form Shannon entropies (nats) of softmax rows, Eq. 1 of the paper.\n")
        f.write("# Row: m entries at c, V-m entries at 0.  H = ln Z - m c e^c / Z, Z = m e^c + V - m.\n")
        f.write("# Written by make_closed_forms.py (60-digit decimal arithmetic; no oracle, no GPU).\n")
        f.write("# kind V m c H\n")
        for kind, V, m, c in CASES:
            f.write(f"{kind} {V} {m} {c} {entropy(V, m, c):.18f}\n")
