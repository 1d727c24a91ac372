"""Writes activation_fixed_points.txt: values of the activation definitions at fixed points,
evaluated with 40-digit arithmetic (mpmath), independent of both the CPU oracle and the CUDA path.

    python tests/golden/make_activation_fixed_points.py

Definitions (the same ones the chains are specified by): sigmoid(z) = 1/(1+e^-z);
gelu_tanh(z) = z/2 * (1 + tanh(sqrt(2/pi) * (z + 0.044715 z^3))); gelu_erf(z) = z/2 * (1 + erf(z/sqrt 2)),
the form the paper's Appendix C.2 listings use.
"""
import os

import mpmath as mp

mp.mp.dps = 40


def sigmoid(z):
    return 1 / (1 + mp.e ** (-z))


def gelu_tanh(z):
    return z / 2 * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (z + mp.mpf("0.044715") * z ** 3)))


def gelu_erf(z):
    return z / 2 * (1 + mp.erf(z / mp.sqrt(2)))


POINTS = [("gelu_tanh", gelu_tanh, ["1", "-1", "2", "-3"]), ("gelu_erf", gelu_erf, ["1", "-3"]),
          ("sigmoid", sigmoid, ["1"])]

if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "activation_fixed_points.txt")
    with open(out, "w") as f:
        f.write("# name z value   -- written by make_activation_fixed_points.py (mpmath, 40 digits;\n"
                "# definitions in that file's docstring; the erf form is the one in the paper's Appendix C.2)\n")
        for name, fn, zs in POINTS:
            for z in zs:
                f.write("%s %s %s\n" % (name, z, mp.nstr(fn(mp.mpf(z)), 20)))
    print(open(out).read())
