"""Pins for the oracle's Cook-Toom construction (Section 3.1, Appendix A.2)."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import wino_inputs as wi

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_counts.json")))


@pytest.mark.parametrize("m", [2, 4, 6])
def test_fir_identity_exact(m):
    # 1-D form of Eq. 1: sum_j AT[i][j] G[j][k] BT[j][l] == [l == i + k]
    ct = oracle.cook_toom(m, wi.POINTS[m])
    t = m + 2
    for i in range(m):
        for k in range(3):
            for l in range(t):
                s = sum(ct["AT"][i, j] * ct["G"][j, k] * ct["BT"][j, l] for j in range(t))
                assert s == (1 if l == i + k else 0), (m, i, k, l, s)


@pytest.mark.parametrize("m", [1, 3, 5])
def test_identity_other_sizes_and_points(m):
    pts = [0, 1, -1, 2, -2, Fraction(1, 2), Fraction(-1, 2)][: m + 1]
    ct = oracle.cook_toom(m, pts)
    t = m + 2
    for i in range(m):
        for k in range(3):
            for l in range(t):
                s = sum(ct["AT"][i, j] * ct["G"][j, k] * ct["BT"][j, l] for j in range(t))
                assert s == (1 if l == i + k else 0)


def test_point_order_permutes_rows():
    a = oracle.cook_toom(2, [0, 1, -1])
    b = oracle.cook_toom(2, [0, -1, 1])
    assert (a["BT"][1] == b["BT"][2]).all() and (a["G"][2] == b["G"][1]).all()


def _zero_fraction(M):
    return Fraction(sum(1 for v in M.flat if v == 0), M.size)


def test_zero_fractions_match_appendix():
    for name, m in (("F2", 2), ("F4", 4)):
        ct = oracle.cook_toom(m, wi.POINTS[m])
        for mat, want in GOLD["zero_fraction"][name].items():
            assert abs(float(_zero_fraction(ct[mat])) - want) < 0.006, (name, mat)
    # the figure that the stated points do not reproduce: document, do not assert equal
    f4 = oracle.cook_toom(4, wi.POINTS[4])
    assert _zero_fraction(f4["BT"]) == Fraction(14, 36)
    assert abs(float(_zero_fraction(f4["BT"])) - GOLD["not_reproduced"]["F4"]["BT"]) > 0.1


def test_weight_expansion():
    assert round(4 * 4 / 9, 2) == GOLD["weight_expansion"]["F2"]
    assert 6 * 6 / 9 == GOLD["weight_expansion"]["F4"]
    # the oracle's transformed-weight buffer has exactly that many bytes per weight byte
    L = oracle.Layer(1, 4, 4, 4, 4, 2, *(oracle.cook_toom(2, wi.POINTS[2])[k] for k in ("BT32", "G32", "AT32")))
    U = oracle.weight_stage(L, np.zeros((4, 3, 3, 4), np.int8))
    assert U.size / (4 * 9 * 4) == 16 / 9


def test_structure_of_default_matrices():
    f2 = oracle.cook_toom(2, wi.POINTS[2])
    f4 = oracle.cook_toom(4, wi.POINTS[4])
    f6 = oracle.cook_toom(6, wi.POINTS[6])
    # F2 / F4: B^T is integer; F2's G and A are built from {0, +-1, +-1/2}
    assert all(v.denominator == 1 for v in f2["BT"].flat)
    assert all(v.denominator == 1 for v in f4["BT"].flat)
    assert {abs(v) for v in f2["G"].flat} == {0, 1, Fraction(1, 2)}
    assert {abs(v) for v in f2["AT"].flat} == {0, 1}
    assert {abs(v) for v in f4["G"].flat} == {0, 1, Fraction(1, 4), Fraction(1, 6), Fraction(1, 12), Fraction(1, 24)}
    assert max(abs(v) for v in f4["AT"].flat) == 8
    # F6: quarter-integers in B^T, powers of two up to 32 and down to 1/32 in A^T
    assert all((v * 4).denominator == 1 for v in f6["BT"].flat)
    assert max(abs(v) for v in f6["AT"].flat) == 32 and Fraction(1, 32) in set(f6["AT"].flat)
    # max row abs-sums quoted in the exactness analysis
    rs = lambda M: max(sum(abs(v) for v in row) for row in M)
    assert (rs(f2["BT"]), rs(f2["AT"])) == (2, 3)
    assert (rs(f4["BT"]), rs(f4["AT"])) == (10, 19)
    assert rs(f6["BT"]) == 15


def _round_f32(fr: Fraction) -> np.float32:
    """Independent correctly rounded Fraction -> binary32 (nearest, ties to even)."""
    c0 = np.float32(fr.numerator / fr.denominator)
    cands = [c0, np.nextafter(c0, np.float32(np.inf)), np.nextafter(c0, np.float32(-np.inf))]
    best = None
    for c in cands:
        err = abs(Fraction(float(c)) - fr)
        even = (int(np.array(c, np.float32).view(np.uint32)) & 1) == 0
        key = (err, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


@pytest.mark.parametrize("m", [2, 4, 6])
def test_fp32_rounding_is_correct(m):
    ct = oracle.cook_toom(m, wi.POINTS[m])
    for k in ("BT", "G", "AT"):
        want = np.array([[_round_f32(v) for v in row] for row in ct[k]], np.float32)
        assert (want.view(np.uint32) == ct[k + "32"].view(np.uint32)).all()
        assert np.allclose(ct[k + "64"], np.array(ct[k], dtype=np.float64), rtol=0, atol=1e-16)
