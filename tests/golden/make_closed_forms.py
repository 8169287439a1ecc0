"""Writes closed_forms.txt: entropies that follow from textbook formulas alone.

Uses only Python's math module (neither the oracle nor the CUDA library), so the
stored values are independent of both sides of every parity test.
"""
import math
import os

HEADER = """# Closed-form entropies (nats) of rows with a textbook distribution; written by
# tests/golden/make_closed_forms.py with Python's math module only (no oracle, no CUDA).
# Eq. 7 of the paper uses H of the draft distribution; a uniform row over V tokens has H = ln V.
# kind V L value
"""


def spike(V, L):
    # one logit L above V-1 zeros: a = e^L/(e^L+V-1), b = 1/(e^L+V-1)
    a = math.exp(L) / (math.exp(L) + V - 1)
    b = 1.0 / (math.exp(L) + V - 1)
    return -(a * math.log(a) + (V - 1) * b * math.log(b))


def main():
    lines = [HEADER]
    for V in (8, 32000, 152064, 256000):
        lines.append("uniform %d 0 %.17g\n" % (V, math.log(V)))
    for V in (8, 32000, 152064, 256000):
        for L in (1.0, 5.0, 12.0, 20.0):
            lines.append("spike %d %.1f %.17g\n" % (V, L, spike(V, L)))
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt"), "w") as f:
        f.writelines(lines)


if __name__ == "__main__":
    main()
