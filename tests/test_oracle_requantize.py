"""Pins for the oracle's output quantizer on direct-convolution accumulators
(``requantize_acc``: the uniform per-layer quantizer of Section 5.1 applied to
the lossless candidate of Section 4, with the optional real-valued bias) and
for the float-output path of the Winograd layer, on whole tensors.

Three independent pins: a hand-worked table (ties, saturation, zero points,
bias), an exact-rational recomputation on random vectors (the fused
multiply-add rounds once to binary32, then the result is rounded half to even),
and the end-to-end identity "scale 1, no bias: codes are the clamped
accumulators"."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
import wino_inputs as wi
from oracle import Quant

from helpers import build_layer

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "requantize_table.json")))


def _round_f32(fr: Fraction) -> Fraction:
    """Correctly rounded Fraction -> binary32 (nearest, ties to even), as a Fraction.
    Works on the integer significand, so it shares nothing with numpy's conversions."""
    if fr == 0:
        return Fraction(0)
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1                       # now 2^e <= a < 2^(e+1)
    e = max(e, -126)                 # subnormal range shares the exponent of the smallest normal
    ulp = Fraction(2) ** (e - 23)
    q = a / ulp
    fl = q.__floor__()
    rem = q - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return sign * fl * ulp


def _rne(fr: Fraction) -> int:
    fl = fr.__floor__()
    rem = fr - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl


def test_round_f32_helper_agrees_with_known_values():
    # the helper itself, against values whose binary32 neighbours are known by construction
    assert _round_f32(Fraction(1, 3)) == Fraction(11184811, 2 ** 25)       # 0x3EAAAAAB
    assert _round_f32(Fraction(2 ** 24 + 1)) == Fraction(2 ** 24)           # tie -> even
    assert _round_f32(Fraction(2 ** 24 + 3)) == Fraction(2 ** 24 + 4)       # tie -> even
    assert _round_f32(Fraction(-5, 2)) == Fraction(-5, 2)
    for v in (0.1, -3.7, 1e-3, 123456.789):
        assert _round_f32(Fraction(v)) == Fraction(float(np.float32(v)))


@pytest.mark.parametrize("row", GOLD["rows"] + GOLD["rounding_rows"])
def test_requantize_table(row):
    acc, s_in, s_Y, bias, z, qmin, qmax, want = row
    q = Quant(scale=s_Y, zero_point=z, qmin=qmin, qmax=qmax)
    b = None if bias is None else np.array([bias], np.float32)
    got = oracle.requantize_acc(np.array([[acc]], np.int32), s_in, q, b)
    assert int(got[0, 0]) == want


def test_bias_is_indexed_by_output_channel():
    # bias[k] belongs to the innermost index: rows of two channels, +0.5 / -0.5 in code units
    acc = np.array([[1, 1], [2, 2], [4, 3]], np.int32)
    got = oracle.requantize_acc(acc, 1.0, Quant(scale=1.0), np.array([0.5, -0.5], np.float32))
    assert got.tolist() == [[2, 0], [2, 2], [4, 2]]


@pytest.mark.parametrize("seed,relu,z", [(1, False, 0), (2, True, 0), (3, False, -7), (4, False, 11)])
def test_requantize_against_exact_rationals(seed, relu, z):
    K, n = 5, 400
    top = 127 * 127 * 64
    acc = np.floor(wi.uniform(seed, 1, n * K) * (2 * top + 1) - top).astype(np.int32).reshape(n, K)
    u = wi.uniform(seed, 2, 4 + K)
    s_in = float(np.float32(0.001 + 0.002 * u[0])) * float(np.float32(0.0005 + 0.001 * u[1]))
    # an output scale under which roughly a tenth of the codes saturate
    s_Y = float(np.float32(np.abs(acc).max() * s_in / (127 * (1.0 + 0.2 * u[2]))))
    bias = ((u[4:] - 0.5) * 40 * s_Y).astype(np.float32)
    qmin, qmax = (0 if relu else -127), 127
    q = Quant(scale=s_Y, zero_point=z, qmin=qmin, qmax=qmax)
    got = oracle.requantize_acc(acc, s_in, q, bias)
    # the contract's constants, from exact rationals rounded once each
    mult = _round_f32(Fraction(s_in) / Fraction(s_Y))
    bs = [_round_f32(Fraction(float(b)) / Fraction(s_Y)) for b in bias]
    clipped = 0
    for i in range(n):
        for k in range(K):
            yf = _round_f32(Fraction(int(acc[i, k])) * mult + bs[k])   # one fused multiply-add
            want = min(max(_rne(yf) + z, qmin), qmax)
            assert int(got[i, k]) == want, (i, k, int(acc[i, k]), float(yf))
            clipped += want in (qmin, qmax)
    assert 0 < clipped < n * K
    assert len(np.unique(got)) > 50


def test_requantize_identity_scale_one():
    acc = np.floor(wi.uniform(9, 1, 192) * 601 - 300).astype(np.int32).reshape(64, 3)
    got = oracle.requantize_acc(acc, 1.0, Quant(scale=1.0))
    assert (got == np.clip(acc, -127, 127)).all()


def test_direct_conv_pipeline_matches_float_convolution():
    # accumulate + requantize against a double-precision convolution of the real values:
    # codes may differ from the real-valued result by the rounding of the multiplier only
    x_q = wi.uniform_int8(12, 1, (2, 6, 7, 8), 0, 127)
    w_q = wi.uniform_int8(12, 2, (4, 3, 3, 8))
    s_x, s_w = 1.0 / 32, 1.0 / 256
    acc = oracle.direct_conv_i32(x_q, w_q)
    real = oracle.direct_f64(x_q.astype(np.float64) * s_x, w_q.astype(np.float64) * s_w)[0]
    s_Y = float(np.float32(np.abs(real).max() / 127))
    got = oracle.requantize_acc(acc, s_x * s_w, Quant(scale=s_Y)).astype(np.float64)
    scaled = real / s_Y
    assert np.abs(got - scaled).max() <= 0.5 + 1e-4
    assert np.abs(got).max() == 127


# ---------------------------------------------------------------------------
# Float output of the Winograd layer on a whole tensor: y = fmaf(Y, s_acc, bias)
# rounded once, with s_acc = s_M (Q_M on) or s_U * s_V (Q_M off).
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("m,q_M", [(2, True), (4, True), (4, False), (6, True)])
def test_float_output_whole_tensor_exact(m, q_M):
    wl = wi.Workload("tiny", 310 + m, 2, 4, 2 * m + 1, m + 2, 3, m)
    L, x_q, w_q, bias = build_layer(wl, out_dtype=1, q_M=q_M)
    y, d = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    _, Yf = oracle.output_stage(L, d["M"], d["m_q"] if q_M else None, bias, want_f32=True)
    if q_M:
        s_acc = Fraction(float(np.float32(L.q_M.scale)))
    else:
        s_acc = _round_f32(Fraction(float(np.float32(L.q_U.scale))) * Fraction(float(np.float32(L.q_V.scale))))
    checked = 0
    for n in range(L.N):
        for h in range(L.H):
            for w in range(L.W):
                tau = (n * L.TH + h // m) * L.TW + w // m
                for k in range(L.K):
                    Y = Fraction(float(Yf[tau, k, h % m, w % m]))
                    want = _round_f32(Y * s_acc + Fraction(float(bias[k])))
                    assert Fraction(float(y[n, h, w, k])) == want
                    checked += 1
    assert checked == y.size and np.abs(y).max() > 0


def test_per_channel_scales_equal_the_per_layer_quantizer_channel_by_channel():
    """requantize_acc with per-output-channel scales: every channel must equal the per-layer
    quantizer (pinned above) applied to that channel with its own scales; equal scales must
    reproduce the per-layer result."""
    K = 7
    acc = ((wi.bits64(71, 5, 6 * 5 * K) % np.uint64(40001)).astype(np.int64) - 20000).astype(np.int32).reshape(6, 5, K)
    bias = wi.bias_values(71, 3, K, 2.0)
    s_x = np.float32(1 / 32)
    f_w, _, _, f_Y = wi.channel_factors(71, K, 4.0)
    s_w_K = (np.float32(0.003) * f_w).astype(np.float32)
    s_Y_K = (np.float32(0.02) * f_Y).astype(np.float32)
    s_in_K = s_w_K.astype(np.float64) * np.float64(s_x)
    q_Y = Quant(scale=0.02, zero_point=3, qmin=-100, qmax=120)
    got = oracle.requantize_acc(acc, 0.0, q_Y, bias, s_in_K=s_in_K, s_Y_K=s_Y_K)
    for k in range(K):
        q_k = Quant(scale=float(s_Y_K[k]), zero_point=3, qmin=-100, qmax=120)
        want = oracle.requantize_acc(acc[..., k:k + 1], float(s_in_K[k]), q_k, bias[k:k + 1])
        assert (got[..., k] == want[..., 0]).all(), k
    assert len(np.unique(got)) > 20
    s_in = float(np.float64(s_x) * np.float64(np.float32(0.003)))
    same = oracle.requantize_acc(acc, s_in, q_Y, bias, s_in_K=np.full(K, s_in), s_Y_K=np.full(K, 0.02, np.float32))
    assert (same == oracle.requantize_acc(acc, s_in, q_Y, bias)).all()
    only_w = oracle.requantize_acc(acc, s_in, q_Y, bias, s_in_K=s_in_K)
    for k in range(K):
        want = oracle.requantize_acc(acc[..., k:k + 1], float(s_in_K[k]), q_Y, bias[k:k + 1])
        assert (only_w[..., k] == want[..., 0]).all()
