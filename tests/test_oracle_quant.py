"""Pins for the oracle's uniform quantizer (Section 5.1: per-layer symmetric
uniform quantization; round-half-to-even, clamp)."""
import json
import os
from fractions import Fraction

import numpy as np

import oracle
import wino_inputs as wi

TABLE = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "quantizer_table.json")))


def test_rounding_table():
    for v, mult, z, qmin, qmax, want in TABLE["rows"]:
        got = oracle.quantize(np.float32(v), np.float32(mult), z, qmin, qmax)
        assert got == want, (v, mult, z, qmin, qmax, got, want)


def test_against_second_implementation():
    # independent statement: numpy's rint on the exact (float64) product of the two
    # float32 numbers, integer clamp afterwards
    n = 20000
    v = (wi.normal(7, 1, n) * 300).astype(np.float32)
    v[:200] = (np.arange(200) - 100).astype(np.float32) / 2  # exact ties
    mult = np.float32(0.37)
    for z, qmin, qmax in ((0, -127, 127), (3, -127, 127), (0, 0, 127), (-10, -128, 127)):
        prod = v.astype(np.float64) * np.float64(mult)
        want = np.clip(np.rint(prod).astype(np.int64) + z, qmin, qmax)
        got = np.array([oracle.quantize(x, mult, z, qmin, qmax) for x in v])
        assert (got == want).all()


def test_product_is_rounded_once_not_twice():
    # a product that the fp32 multiply would round onto a tie: v * mult = 2.5 + 2^-25
    # exactly; rounding it to fp32 first gives 2.5 -> 2, rounding the exact value gives 3
    v, mult = np.float32(1.25 * (1 + 2.0 ** -23)), np.float32(2.0 * (1 - 2.0 ** -24))
    exact = Fraction(float(v)) * Fraction(float(mult))
    assert exact > Fraction(5, 2) and np.float32(v * mult) == np.float32(2.5)
    assert oracle.quantize(v, mult) == 3
    assert oracle.quantize(-v, mult) == -3


def test_multipliers_are_single_rounded_double_ratios():
    ct = oracle.cook_toom(2, wi.POINTS[2])
    L = oracle.Layer(1, 4, 4, 4, 4, 2, ct["BT32"], ct["G32"], ct["AT32"])
    L.q_x.scale, L.q_w.scale, L.q_V.scale, L.q_U.scale, L.q_M.scale, L.q_Y.scale = (
        0.031, 0.0017, 0.093, 0.0009, 0.011, 0.047)
    f = lambda s: float(np.float32(s))
    mul = oracle.multipliers(L)
    sUV = f(L.q_U.scale) * f(L.q_V.scale)
    want = [f(L.q_x.scale) / f(L.q_V.scale), f(L.q_w.scale) / f(L.q_U.scale),
            sUV / f(L.q_M.scale), f(L.q_M.scale) / f(L.q_Y.scale), f(L.q_M.scale)]
    assert (mul == np.array(want, np.float64).astype(np.float32)).all()
    L.q_M.enabled = 0
    mul = oracle.multipliers(L)
    assert mul[3] == np.float32(sUV / f(L.q_Y.scale)) and mul[4] == np.float32(sUV)
