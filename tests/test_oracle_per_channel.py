"""Pins for the oracle's per-output-channel scales (Section 7 names per-channel quantization
as the step beyond the per-layer scales of Section 5.1).  The per-layer pipeline is pinned
elsewhere (exact rationals, lossless F2, hand tables); here the per-channel form is tied to
it: equal scales must reproduce it, and each output channel must equal the per-layer
pipeline run on that channel alone with that channel's scales."""
import copy

import numpy as np
import pytest

import oracle
import wino_inputs as wi
from helpers import build_layer, per_channel


def _layer(m, seed, q_M=True, out_dtype=0, K=5):
    wl = wi.Workload("pc", seed, 2, 6, 2 * m + 1, m + 2, K, m)
    return build_layer(wl, q_M=q_M, out_dtype=out_dtype)


@pytest.mark.parametrize("m", [2, 4, 6])
def test_equal_channel_scales_reduce_to_the_per_layer_pipeline(m):
    L, x_q, w_q, bias = _layer(m, 900 + m)
    P = copy.deepcopy(L)
    P.s_w_K = np.full(L.K, L.q_w.scale, np.float32)
    P.s_U_K = np.full(L.K, L.q_U.scale, np.float32)
    P.s_M_K = np.full(L.K, L.q_M.scale, np.float32)
    P.s_Y_K = np.full(L.K, L.q_Y.scale, np.float32)
    y0, d0 = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    y1, d1 = oracle.forward(P, x_q, w_q, bias=bias, dumps=True)
    assert (y0 == y1).all()
    for k in d0:
        assert (d0[k] == d1[k]).all(), k


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("variant", ["int8", "no_qm", "float_out", "no_qm_float"])
def test_each_channel_equals_the_per_layer_pipeline_on_that_channel(m, variant):
    q_M = variant in ("int8", "float_out")
    out_dtype = 1 if "float" in variant else 0
    L, x_q, w_q, bias = _layer(m, 910 + m, q_M=q_M, out_dtype=out_dtype)
    P = per_channel(L, 33 + m, spread=3.0)
    y, d = oracle.forward(P, x_q, w_q, bias=bias, dumps=True)
    changed = 0
    y_plain = oracle.forward(L, x_q, w_q, bias=bias)
    for k in range(L.K):
        S = copy.deepcopy(L)          # one-filter layer with channel k's scales as layer scales
        S.K = 1
        S.q_w.scale = float(P.s_w_K[k])
        S.q_U.scale = float(P.s_U_K[k])
        if q_M:
            S.q_M.scale = float(P.s_M_K[k])
        S.q_Y.scale = float(P.s_Y_K[k])
        yk, dk = oracle.forward(S, x_q, w_q[k:k + 1], bias=bias[k:k + 1], dumps=True)
        assert (d["U_q"][:, k] == dk["U_q"][:, 0]).all()
        assert (d["M"][:, :, k] == dk["M"][:, :, 0]).all()
        if q_M:
            assert (d["m_q"][:, :, k] == dk["m_q"][:, :, 0]).all()
        assert (y[..., k] == yk[..., 0]).all()
        changed += int((y[..., k] != y_plain[..., k]).any())
    assert (d["V_q"] == oracle.input_stage(L, x_q)).all()     # the input side has no channel scale
    assert changed >= L.K - 1                                   # the scales did take effect


def test_stage_functions_follow_the_channel_scales_too():
    L, x_q, w_q, bias = _layer(4, 950)
    P = per_channel(L, 5)
    y, d = oracle.forward(P, x_q, w_q, bias=bias, dumps=True)
    Uq = oracle.weight_stage(P, w_q)
    M = oracle.hadamard(P, d["V_q"], Uq)
    mq = oracle.quantize_M(P, M)
    assert (Uq == d["U_q"]).all() and (M == d["M"]).all() and (mq == d["m_q"]).all()
    assert (oracle.output_stage(P, M, mq, bias) == y).all()


@pytest.mark.parametrize("q_M", [False, True])
def test_power_of_two_rescaling_of_one_channel_leaves_its_codes_unchanged(q_M):
    """Multiplying every scale of channel k (s_w, s_U, s_M, s_Y) and bias[k] by 2^j rescales
    channel k's real values exactly, so every code of the layer stays what it was."""
    L, x_q, w_q, bias = _layer(4, 960, q_M=q_M)
    P = per_channel(L, 6)
    Q = copy.deepcopy(P)
    b2 = bias.copy()
    for k, j in ((1, 3), (3, -2)):
        for name in ("s_w_K", "s_U_K", "s_M_K", "s_Y_K"):
            if getattr(Q, name) is not None:
                getattr(Q, name)[k] *= 2.0 ** j
        b2[k] *= 2.0 ** j
    y0, d0 = oracle.forward(P, x_q, w_q, bias=bias, dumps=True)
    y1, d1 = oracle.forward(Q, x_q, w_q, bias=b2, dumps=True)
    assert (d0["U_q"] == d1["U_q"]).all() and (d0["M"] == d1["M"]).all()
    assert (d0["m_q"] == d1["m_q"]).all()
    assert (y0 == y1).all()


def test_channel_scales_recover_filters_of_small_norm():
    """What per-channel scales are for (Section 7): filters whose norms differ.  Real weights
    with gains spread over a factor of 64 are quantized once with one scale and once with one
    scale per filter; against the double-precision convolution of the real tensors, the
    low-gain channels come out several times more accurate with per-channel scales, and the
    high-gain ones no worse."""
    from helpers import matrices
    from oracle import Layer, Quant
    from oracle.calibrate import calibrate, calibrate_per_channel
    m, N, C, H, W, K = 2, 2, 16, 8, 8, 12
    x_q = wi.halfnormal_codes(321, wi.S_X, (N, H, W, C))
    s_x = np.float32(1.0 / 32.0)
    gains = np.float64(2.0) ** (-(np.arange(K) % 7))              # 1 ... 1/64
    w_real = wi.normal(321, wi.S_W, K * 9 * C).reshape(K, 3, 3, C) * 0.05 * gains[:, None, None, None]
    BT, G, AT = matrices(m)
    ref = oracle.direct_f64(x_q.astype(np.float64) * float(s_x), w_real, pad=1)[0]

    def rel_err(y, ks):
        return float(np.sqrt(np.mean((y[..., ks] - ref[..., ks]) ** 2) / np.mean(ref[..., ks] ** 2)))

    base = Layer(N, C, H, W, K, m, BT, G, AT, out_dtype=1)
    base.q_x = Quant(scale=float(s_x))
    # one scale for all filters
    s_w = np.float32(np.abs(w_real).max() / 127.0)
    w_q1 = np.clip(np.rint(w_real / np.float64(s_w)), -127, 127).astype(np.int8)
    L1 = copy.deepcopy(base)
    L1.q_w = Quant(scale=float(s_w))
    L1 = calibrate(L1, x_q, w_q1)
    y1 = oracle.forward(L1, x_q, w_q1)
    # one scale per filter
    s_wk = (np.abs(w_real).max(axis=(1, 2, 3)) / 127.0).astype(np.float32)
    w_q2 = np.clip(np.rint(w_real / s_wk.astype(np.float64)[:, None, None, None]), -127, 127).astype(np.int8)
    L2 = copy.deepcopy(base)
    L2.s_w_K = s_wk
    L2 = calibrate_per_channel(L2, x_q, w_q2, output_per_channel=True)
    y2 = oracle.forward(L2, x_q, w_q2)
    low = [k for k in range(K) if gains[k] <= 1.0 / 16]
    high = [k for k in range(K) if gains[k] == 1.0]
    assert rel_err(y1, low) > 4 * rel_err(y2, low), (rel_err(y1, low), rel_err(y2, low))
    assert rel_err(y2, high) < 1.5 * rel_err(y1, high) + 1e-3
    assert rel_err(y2, list(range(K))) < 0.05
