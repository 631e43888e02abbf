"""Writes gelu_tanh_values.txt: the tanh form of GELU,

    G(x) = 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))),

evaluated with 50-digit decimal arithmetic (tanh from the exponential series of the `decimal`
module, pi from Machin's formula), so the stored values depend on no floating-point library.
The formula is this library's problem statement (the paper has no GELU); the values pin the
oracle's activation.  Run: python tests/golden/make_gelu_tanh_values.py
"""
import os
from decimal import Decimal, getcontext

getcontext().prec = 50


def arctan_inv(n: int) -> Decimal:
    """atan(1/n) by its Taylor series."""
    x = Decimal(1) / n
    term, total, k, x2 = x, x, 1, x * x
    while abs(term) > Decimal(10) ** -48:
        term = -term * x2
        k += 2
        total += term / k
    return total


PI = 4 * (4 * arctan_inv(5) - arctan_inv(239))


def tanh(u: Decimal) -> Decimal:
    e = (2 * u).exp()
    return (e - 1) / (e + 1)


def gelu(x: Decimal) -> Decimal:
    c = (Decimal(2) / PI).sqrt()
    return Decimal("0.5") * x * (1 + tanh(c * (x + Decimal("0.044715") * x ** 3)))


if __name__ == "__main__":
    xs = ["0", "0.5", "-0.5", "1", "-1", "2", "-2", "3", "-3", "6", "-6", "0.125", "-0.75", "1.5"]
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "gelu_tanh_values.txt")
    with open(path, "w") as f:
        f.write("# x  G(x) = 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))), 30 significant digits\n")
        f.write("# written by make_gelu_tanh_values.py (50-digit decimal arithmetic, no floating-point library)\n")
        for x in xs:
            g = gelu(Decimal(x))
            f.write(f"{x} {g:.30e}\n")
    print(open(path).read())
