"""Writes activation_closed_forms.txt: SiLU and GELU-tanh at fixed points from their closed
forms, evaluated with 60-digit arithmetic (mpmath) and printed to 20 significant digits.
Calls neither the oracle nor the CUDA path.

  silu(x)      = x / (1 + e^-x)
  gelu_tanh(x) = x/2 * (1 + tanh( sqrt(2/pi) * (x + 0.044715 x^3) ))
  gelu_erf(x)  = x/2 * (1 + erf(x / sqrt 2))      sigmoid(x) = 1 / (1 + e^-x)
  tanh(x)                                          leaky_relu(x) = x if x > 0 else x/100
"""
import os

import mpmath as mp

mp.mp.dps = 60
POINTS = ["-10", "-3", "-2", "-1", "-0.5", "0", "0.5", "1", "2", "3", "10"]


def silu(x):
    return x / (1 + mp.e ** (-x))


def gelu_tanh(x):
    return x / 2 * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (x + mp.mpf("0.044715") * x ** 3)))


def gelu_erf(x):
    return x / 2 * (1 + mp.erf(x / mp.sqrt(2)))


def sigmoid(x):
    return 1 / (1 + mp.e ** (-x))


def leaky_relu(x):
    return x if x > 0 else x / 100


here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "activation_closed_forms.txt"), "w") as f:
    f.write("# act x value   (closed forms at 60 digits, see make_activation_golden.py; the paper prints no values)\n")
    for name, fn in (("silu", silu), ("gelu_tanh", gelu_tanh), ("gelu_erf", gelu_erf), ("sigmoid", sigmoid),
                     ("tanh", mp.tanh), ("leaky_relu", leaky_relu)):
        for p in POINTS:
            f.write(f"{name} {p} {mp.nstr(fn(mp.mpf(p)), 20)}\n")
