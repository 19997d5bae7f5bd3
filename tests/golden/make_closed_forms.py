"""Writes closed_forms.txt: the four activations and their derivatives at 50 digits.

    python tests/golden/make_closed_forms.py

The values come from the LITERAL definitions -- Table I of the paper for GELU (tanh form),
Swish and Mish, x * Phi(x) for the erf form that the paper cites -- evaluated with mpmath at 50
digits and differentiated numerically by mpmath (mp.diff), never from the oracle: the file is a
pin FOR the oracle.  Stored with 20 significant digits.  Rows:
  table     f and f' on a grid that reaches into both tails
  extremum  the stationary points of f' (roots of f'') and f' there; for the erf form
            f'' = phi(x) (2 - x^2), so they sit at +-sqrt(2) exactly
  root      the sign change of f' on the negative axis; for Swish f(root) = root + 1 there,
            since f' = s + x s (1 - s) = 0 gives x (1 - s) = -1, i.e. x s = x + 1
The constant 0.044715 is taken as the decimal the paper prints.
"""
import os

import mpmath as mp

mp.mp.dps = 50
A = mp.mpf("0.044715")


def gelu_erf(x):
    return x * (1 + mp.erf(x / mp.sqrt(2))) / 2


def gelu_tanh(x):
    return x / 2 * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (x + A * x ** 3)))


def swish(x):
    return x / (1 + mp.exp(-x))


def mish(x):
    return x * mp.tanh(mp.log(1 + mp.exp(x)))


F = {"gelu_erf": gelu_erf, "gelu_tanh": gelu_tanh, "swish": swish, "mish": mish}
GRID = {"gelu_erf": (-10, -5, -3, -1, -0.5, 0.5, 1, 3, 5), "gelu_tanh": (-10, -5, -3, -1, -0.5, 0.5, 1, 3, 5),
        "swish": (-80, -20, -10, -5, -3, -1, -0.5, 0.5, 1, 3, 5, 10), "mish": (-80, -20, -10, -5, -3, -1, -0.5, 0.5, 1, 3, 5, 10)}
EXTREMA = {"gelu_erf": (1.4, -1.4), "gelu_tanh": (1.4, -1.4), "swish": (2.4, -2.4), "mish": (1.5, -2.25)}
ROOTS = {"gelu_erf": -0.75, "gelu_tanh": -0.75, "swish": -1.28, "mish": -1.19}


def s(v):
    return mp.nstr(v, 20, min_fixed=-1, max_fixed=1, strip_zeros=False)


def d1(f, x):
    # mp.diff at the working precision loses half the digits: evaluate it with 100 more
    with mp.workdps(150):
        return mp.diff(f, mp.mpf(x))


def main():
    lines = ["# Written by make_closed_forms.py (mpmath %s, 50 digits) from the literal definitions: Table I of the" % mp.__version__,
             "# paper (GELU tanh form, Swish, Mish) and x*Phi(x) (GELU erf form); derivatives by mp.diff.",
             "# columns: row-kind  activation  x  f(x)  f'(x)"]
    for kind, f in F.items():
        for x in GRID[kind]:
            lines.append(f"table {kind} {s(mp.mpf(x))} {s(f(mp.mpf(x)))} {s(d1(f, x))}")
    for kind, f in F.items():
        for guess in EXTREMA[kind]:
            with mp.workdps(120):
                x = mp.findroot(lambda t: mp.diff(f, t, 2), mp.mpf(guess))
            lines.append(f"extremum {kind} {s(x)} {s(f(x))} {s(d1(f, x))}")
    for kind, f in F.items():
        with mp.workdps(120):
            x = mp.findroot(lambda t: mp.diff(f, t), mp.mpf(ROOTS[kind]))
        lines.append(f"root {kind} {s(x)} {s(f(x))} 0")
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt")
    with open(path, "w") as out:
        out.write("\n".join(lines) + "\n")
    print(path, len(lines) - 3, "rows")


if __name__ == "__main__":
    main()
