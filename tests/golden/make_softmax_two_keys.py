"""Writes softmax_two_keys.txt: the closed-form softmax over the two scores (0, 1)."""
import math
import os

w0 = 1.0 / (1.0 + math.e)
w1 = math.e / (1.0 + math.e)
lse = math.log(1.0 + math.e)
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "softmax_two_keys.txt"), "w") as fh:
    fh.write(f"{w0!r} {w1!r} {lse!r}\n")
    fh.write("# w0 = 1/(1+e), w1 = e/(1+e), lse = ln(1+e): textbook softmax over scores (0, 1).\n")
    fh.write("# The paper prints no worked example of attention; this closed form stands in for one.\n")
