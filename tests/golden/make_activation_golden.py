"""Writes activation_closed_forms.txt: SiLU and GELU-tanh at fixed points from their closed
forms, evaluated with 60-digit arithmetic (mpmath) and printed to 20 significant digits.
Calls neither the oracle nor the CUDA path.

  silu(x)      = x / (1 + e^-x)
  gelu_tanh(x) = x/2 * (1 + tanh( sqrt(2/pi) * (x + 0.044715 x^3) ))
"""
import os

import mpmath as mp

mp.mp.dps = 60
POINTS = ["-10", "-3", "-2", "-1", "-0.5", "0", "0.5", "1", "2", "3", "10"]


def silu(x):
    return x / (1 + mp.e ** (-x))


def gelu_tanh(x):
    return x / 2 * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (x + mp.mpf("0.044715") * x ** 3)))


here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "activation_closed_forms.txt"), "w") as f:
    f.write("# act x value   (closed forms at 60 digits, see make_activation_golden.py; the paper prints no values)\n")
    for name, fn in (("silu", silu), ("gelu_tanh", gelu_tanh)):
        for p in POINTS:
            f.write(f"{name} {p} {mp.nstr(fn(mp.mpf(p)), 20)}\n")
