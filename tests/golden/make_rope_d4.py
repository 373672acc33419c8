"""Writes rope_d4.txt: the 4x4 rotation printed before Eq. 2, multiplied out with math.cos/math.sin only.

No oracle or library code is called: theta_0 = base^0 = 1, theta_1 = base^(-2/4); the vector (x0,x1,x2,x3) is
rotated pairwise, (x0,x1) by m*theta_0 and (x2,x3) by m*theta_1, exactly as the printed matrix reads.
"""
import math
import os

cases = [(10000.0, 3, (1.0, 2.0, 3.0, 4.0)), (10000.0, 517, (-0.5, 0.25, 2.0, -1.0)), (500000.0, 32256, (1.0, 0.0, 0.0, 1.0))]
lines = ["# base m x0 x1 x2 x3 -> y0 y1 y2 y3 ; y = R_{Theta,m} x for D=4, adjacent pairs (matrix before Eq. 2)"]
for base, m, x in cases:
    th = [1.0, base ** (-2.0 / 4.0)]
    y = []
    for i in range(2):
        c, s = math.cos(m * th[i]), math.sin(m * th[i])
        a, b = x[2 * i], x[2 * i + 1]
        y += [c * a - s * b, s * a + c * b]
    lines.append(" ".join(repr(v) for v in (base, m) + x + tuple(y)))
with open(os.path.join(os.path.dirname(__file__), "rope_d4.txt"), "w") as f:
    f.write("\n".join(lines) + "\n")
