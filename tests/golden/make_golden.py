"""Writes tests/golden/worked_example_g0_2.txt.  Calls only the oracle (exact rationals)."""
import os
import sys
from fractions import Fraction

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import literal  # noqa: E402

G0 = 2
C = (0, 1, 2, 0)
CAP = (3, 3, 3, 3)


def main() -> None:
    ab = [literal.posterior(1, 1, c, G0) for c in C]
    lines = [
        "# Worked example: G0 = 2, uniform Beta(1,1) prior, Phase-A counts c = (0,1,2,0), cap = 3 each.",
        "# Written by make_golden.py from oracle/literal.py (Algorithm 1 Phase B on exact rationals,",
        "# ties to the lowest prompt index).  Columns: B | Delta_1..Delta_4 | objective sum_i U_i(Delta_i)",
    ]
    for B in range(0, sum(CAP) + 1):
        d = literal.greedy(ab, CAP, B)
        obj = literal.objective(ab, d)
        lines.append(f"{B} | {' '.join(map(str, d))} | {obj.numerator}/{obj.denominator}")
    rows = [
        "# Gain rows g(1..5) per class (exact):",
    ]
    for c in (0, 1, 2):
        a, b = literal.posterior(1, 1, c, G0)
        ms = literal.marginals(a, b, 5)
        rows.append(f"# c={c}: " + " ".join(f"{Fraction(m).numerator}/{Fraction(m).denominator}" for m in ms))
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_example_g0_2.txt")
    with open(out, "w") as f:
        f.write("\n".join(lines + rows) + "\n")
    print(out)


if __name__ == "__main__":
    main()
