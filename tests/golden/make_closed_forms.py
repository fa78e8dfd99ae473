"""Writes tests/golden/closed_forms.txt from first principles (math module only).

Two-token closed form for rotary attention (the paper prints no worked
example, so the fixture is a hand-derivable case of the definition):

  case A: head_dim 2, axis T only, theta arbitrary (omega_0 = 1).
          q = (1, 0) at t=0; keys (1, 0) at t=0 and (1, 0) at t=1.
          k~_1 = (cos 1, sin 1), scores = [1, cos 1] / sqrt(2).
  case B: head_dim 4, d_T = 4, theta = 10000: second pair rotates with
          omega_1 = theta ** (-2/4) = 0.01.  q = (0, 0, 1, 0) at t = 0,
          keys (0, 0, 1, 0) at t = 0 and t = 50 -> k~ = (0,0,cos .5, sin .5),
          scores = [1, cos 0.5] / sqrt(4).
  case C: same as B with the query at t = 7: relative angle (50-7)*0.01.

Values are softmax weights w0, w1; the output is w0*v0 + w1*v1.
"""
import math
import os


def softmax2(a, b):
    m = max(a, b)
    ea, eb = math.exp(a - m), math.exp(b - m)
    return ea / (ea + eb), eb / (ea + eb)


lines = ["# name w0 w1   (see make_closed_forms.py for the derivation)"]
w = softmax2(1.0 / math.sqrt(2.0), math.cos(1.0) / math.sqrt(2.0))
lines.append("A %.17g %.17g" % w)
w = softmax2(1.0 / 2.0, math.cos(0.5) / 2.0)
lines.append("B %.17g %.17g" % w)
w = softmax2(math.cos(0.07) / 2.0, math.cos(0.43) / 2.0)
lines.append("C %.17g %.17g" % w)
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt"), "w") as f:
    f.write("\n".join(lines) + "\n")
