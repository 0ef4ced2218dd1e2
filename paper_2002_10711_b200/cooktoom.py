"""Cook-Toom transform matrices for F(m x m, 3 x 3) (paper: Section 3.1).

The library takes B^T, G, A^T as data; this helper produces the default ones
for a set of polynomial points, in exact rational arithmetic, rounded once to
fp32.  Convention: rows of B^T are the monic polynomials prod_{k != j}(x - a_k),
G carries the normalisation 1 / prod_{k != j}(a_j - a_k), the last row belongs
to the point at infinity, and a row whose first G entry is negative is negated
in both B^T and G.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

STANDARD_POINTS = {
    2: [0, 1, -1],
    4: [0, 1, -1, 2, -2],
    6: [0, 1, -1, 2, -2, Fraction(1, 2), Fraction(-1, 2)],
}


def _poly_mul_linear(p, a):
    q = [Fraction(0)] * (len(p) + 1)
    for i, c in enumerate(p):
        q[i + 1] += c
        q[i] -= c * a
    return q


def cook_toom_exact(m: int, points=None):
    """Returns (BT, G, AT) as nested lists of Fractions."""
    t = m + 2
    pts = [Fraction(v) for v in (points if points is not None else STANDARD_POINTS[m])]
    if len(pts) != t - 1 or len(set(pts)) != len(pts):
        raise ValueError("need m+1 distinct finite points")
    BT = [[Fraction(0)] * t for _ in range(t)]
    G = [[Fraction(0)] * 3 for _ in range(t)]
    AT = [[Fraction(0)] * t for _ in range(m)]
    for j, aj in enumerate(pts):
        poly, norm = [Fraction(1)], Fraction(1)
        for k, ak in enumerate(pts):
            if k != j:
                poly = _poly_mul_linear(poly, ak)
                norm *= aj - ak
        sign = -1 if (Fraction(1) / norm) < 0 else 1
        for c, v in enumerate(poly):
            BT[j][c] = sign * v
        for k in range(3):
            G[j][k] = sign * aj ** k / norm
        for i in range(m):
            AT[i][j] = aj ** i
    poly = [Fraction(1)]
    for ak in pts:
        poly = _poly_mul_linear(poly, ak)
    for c, v in enumerate(poly):
        BT[t - 1][c] = v
    G[t - 1][2] = Fraction(1)
    AT[m - 1][t - 1] = Fraction(1)
    return BT, G, AT


def _round_f32(fr: Fraction) -> np.float32:
    """Nearest binary32 to a rational, ties to even."""
    c0 = np.float32(fr.numerator / fr.denominator)
    best = None
    for c in (c0, np.nextafter(c0, np.float32(np.inf)), np.nextafter(c0, np.float32(-np.inf))):
        odd = int(np.array(c, np.float32).view(np.uint32)) & 1
        key = (abs(Fraction(float(c)) - fr), odd)
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def cook_toom(m: int, points=None):
    """Returns (BT, G, AT) as fp32 numpy arrays of shapes [t,t], [t,3], [m,t]."""
    return tuple(np.array([[_round_f32(v) for v in row] for row in M], np.float32)
                 for M in cook_toom_exact(m, points))
