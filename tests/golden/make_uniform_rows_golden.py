"""Writes uniform_rows_scores.txt: exact A2SF scores for uniform attention rows.

With Q = 0 every causal softmax row is uniform, P[i][j] = 1/(i+1) for j <= i, so
Eq. 5 of the paper (0-based: S_j = sum_{i>=j} alpha^(n-1-i) P[i][j]) has the exact
rational value sum_{i=j}^{n-1} alpha^(n-1-i)/(i+1).  Computed here with exact
fractions; no oracle or CUDA code is involved.

Run:  python tests/golden/make_uniform_rows_golden.py
"""
from fractions import Fraction
from pathlib import Path

CASES = [(8, Fraction(1, 2)), (8, Fraction(1)), (8, Fraction(0)), (12, Fraction(3, 10))]


def scores(n, alpha):
    out = []
    for j in range(n):
        s = Fraction(0)
        for i in range(j, n):
            w = Fraction(1) if i == n - 1 else alpha ** (n - 1 - i)
            s += w * Fraction(1, i + 1)
        out.append(s)
    return out


def main():
    lines = ["# n alpha_num alpha_den j score_num score_den   (Eq. 5 with uniform rows, exact)"]
    for n, a in CASES:
        for j, s in enumerate(scores(n, a)):
            lines.append(f"{n} {a.numerator} {a.denominator} {j} {s.numerator} {s.denominator}")
    Path(__file__).with_name("uniform_rows_scores.txt").write_text("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
