"""Writes tests/golden/eckart_young.txt: closed-form truncation errors of the synthetic weight spectra.

For singular values sigma_i = i^-p, i = 1..n, the best rank-r approximation leaves
    ||W - W_r||_F^2 = sum_{i > r} sigma_i^2          (Eckart-Young)
and the relative error of the appendix "Reconstruction Error of Matrix SVD" is
    epsilon = sqrt(sum_{i > r} sigma_i^2 / sum_i sigma_i^2).
The sums are taken directly in fp64, smallest terms first.  Run from the repository root:
    python tests/golden/make_eckart_young.py
"""
import math
import os

CASES = [(128, 0.8, (32,)), (1024, 0.8, (128, 256, 384, 416, 512, 928)), (1024, 0.7, (352, 864))]


def tail(n, p, r):
    return math.fsum(float(i) ** (-2.0 * p) for i in range(n, r, -1))


def main():
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "eckart_young.txt")
    with open(out, "w") as f:
        f.write("# Squared Frobenius tail and relative error of the rank-r truncation of a matrix with singular values\n")
        f.write("# i^-p, i = 1..n (Eckart-Young; epsilon as in the appendix \"Reconstruction Error of Matrix SVD\").\n")
        f.write("# Written by tests/golden/make_eckart_young.py (direct fp64 summation).\n")
        f.write("# columns: n  p  r  tail_sq  epsilon\n")
        for n, p, ranks in CASES:
            total = tail(n, p, 0)
            for r in ranks:
                t = tail(n, p, r)
                f.write(f"{n} {p} {r} {t:.12e} {math.sqrt(t / total):.12e}\n")


if __name__ == "__main__":
    main()
