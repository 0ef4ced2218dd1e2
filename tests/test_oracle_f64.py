"""Un-quantized double-precision Winograd (Eq. 1) against direct convolution,
and the multiplication counts the paper quotes (Sections 1 and 3.1)."""
import json
import os

import numpy as np
import pytest

import oracle
import wino_inputs as wi

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_counts.json")))


def _rand(seed, shape):
    return wi.normal(seed, 11, int(np.prod(shape))).reshape(shape)


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("hw", [(8, 8), (7, 9), (13, 5), (1, 1), (2, 3)])
@pytest.mark.parametrize("pad", [0, 1])
def test_winograd_equals_direct(m, hw, pad):
    H, W = hw
    if pad == 0 and (H < 3 or W < 3):
        pytest.skip("no valid output")
    ct = oracle.cook_toom(m, wi.POINTS[m])
    x = _rand(100 + m, (2, H, W, 3))
    w = _rand(200 + m, (4, 3, 3, 3))
    yw, _ = oracle.winograd_f64(x, w, m, ct["BT64"], ct["G64"], ct["AT64"], pad=pad)
    yd, _ = oracle.direct_f64(x, w, pad=pad)
    assert yw.shape == yd.shape
    assert np.max(np.abs(yw - yd)) < 1e-10


def test_direct_f64_against_numpy_definition():
    x = _rand(1, (1, 5, 6, 2))
    w = _rand(2, (3, 3, 3, 2))
    yd, _ = oracle.direct_f64(x, w, pad=1)
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    want = np.zeros_like(yd)
    for a in range(3):
        for b in range(3):
            want += np.einsum("nhwc,kc->nhwk", xp[:, a:a + 5, b:b + 6, :], w[:, a, b, :])
    assert np.max(np.abs(want - yd)) < 1e-12


def test_multiply_counts_32x32():
    x = _rand(3, (1, 32, 32, 1))
    w = _rand(4, (1, 3, 3, 1))
    ct = oracle.cook_toom(2, wi.POINTS[2])
    _, mw = oracle.winograd_f64(x, w, 2, ct["BT64"], ct["G64"], ct["AT64"], pad=0)
    _, md = oracle.direct_f64(x, w, pad=0)
    assert md == GOLD["mults_32x32_valid"]["direct"]
    assert mw == GOLD["mults_32x32_valid"]["F2"]


@pytest.mark.parametrize("m,key", [(2, "F2"), (4, "F4")])
def test_multiplies_per_output(m, key):
    H = W = 4 * m  # divides evenly: no edge waste
    x = _rand(5, (1, H, W, 1))
    w = _rand(6, (1, 3, 3, 1))
    ct = oracle.cook_toom(m, wi.POINTS[m])
    _, mw = oracle.winograd_f64(x, w, m, ct["BT64"], ct["G64"], ct["AT64"], pad=1)
    _, md = oracle.direct_f64(x, w, pad=1)
    assert md / (H * W) == GOLD["mults_per_output"]["direct"]
    assert mw / (H * W) == GOLD["mults_per_output"][key]


def test_transposed_matrix_is_caught():
    # planting a mistake in the oracle's inputs (B instead of B^T) must break the identity
    ct = oracle.cook_toom(4, wi.POINTS[4])
    x = _rand(7, (1, 8, 8, 2))
    w = _rand(8, (2, 3, 3, 2))
    yd, _ = oracle.direct_f64(x, w)
    yw, _ = oracle.winograd_f64(x, w, 4, ct["BT64"].T.copy(), ct["G64"], ct["AT64"])
    assert np.max(np.abs(yw - yd)) > 1e-3
