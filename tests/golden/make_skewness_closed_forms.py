"""Recomputes the 'expected' column of skewness_closed_forms.txt from the closed forms stated in
that file's comments, in exact rational arithmetic up to the final square roots (no oracle, no
CUDA).  Run by hand; prints the rows."""
import math
from fractions import Fraction


def twopoint(n: int, a: int) -> float:
    m2 = Fraction(a * (n - a), n)
    m3 = Fraction(a * (n - a) * (n - 2 * a), n * n)
    return n / ((n - 1) * (n - 2)) * float(m3) / (float(m2) / (n - 1)) ** 1.5


if __name__ == "__main__":
    for n in (4, 9, 576, 7290):
        print("onehot", n, 1, repr(math.sqrt(n)))
    for n, a in ((10, 3), (100, 5)):
        print("twopoint", n, a, repr(twopoint(n, a)))
    print("symmetric", 7, 0, 0.0)
