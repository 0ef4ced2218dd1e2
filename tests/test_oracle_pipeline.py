"""Pins for the oracle's staged quantized pipeline (Eq. 1 with the quantizers of
Fig. 2): a lossless special case that must equal integer direct convolution, an
exact-rational recomputation on tiny layers, exactness of the Cook-Toom
transforms on integer codes, and invariants."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
import wino_inputs as wi
from oracle import Layer, Quant

from helpers import build_layer, matrices, small


# ---------------------------------------------------------------------------
# F2 lossless special case: with |x| <= 31, |w| <= 14, mult_V = 1, mult_U = 4,
# no Q_M and a float output, no stage rounds or clips, so the pipeline reduces
# to the textbook integer convolution.
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [(2, 8, 8, 8, 4), (1, 64, 5, 7, 3), (3, 3, 1, 1, 2), (1, 16, 9, 4, 16)])
def test_f2_lossless_equals_direct(shape):
    N, C, H, W, K = shape
    BT, G, AT = matrices(2)
    x_q = wi.uniform_int8(21, 1, (N, H, W, C), -31, 31)
    w_q = wi.uniform_int8(21, 2, (K, 3, 3, C), -14, 14)
    L = Layer(N, C, H, W, K, 2, BT, G, AT, out_dtype=1)
    L.q_x = Quant(1.0); L.q_w = Quant(1.0); L.q_V = Quant(1.0); L.q_U = Quant(0.25)
    L.q_M = Quant(enabled=0)
    y, d = oracle.forward(L, x_q, w_q, dumps=True)
    acc = oracle.direct_conv_i32(x_q, w_q)
    assert np.abs(d["V_q"]).max() <= 124 and np.abs(d["U_q"]).max() <= 126
    assert (y == acc.astype(np.float32)).all()
    assert np.abs(acc).max() > 0


def test_direct_conv_i32_against_numpy():
    x_q = wi.uniform_int8(5, 1, (2, 6, 5, 3))
    w_q = wi.uniform_int8(5, 2, (4, 3, 3, 3))
    for stride in (1, 2):
        acc = oracle.direct_conv_i32(x_q, w_q, z_x=2, z_w=-1, stride=stride)
        xp = np.pad(x_q.astype(np.int64) - 2, ((0, 0), (1, 1), (1, 1), (0, 0)))
        want = np.zeros((2, 6, 5, 4), np.int64)
        for a in range(3):
            for b in range(3):
                want += np.einsum("nhwc,kc->nhwk", xp[:, a:a + 6, b:b + 5, :], w_q[:, a, b, :].astype(np.int64) + 1)
        assert (acc == want[:, ::stride, ::stride, :]).all()


# ---------------------------------------------------------------------------
# Cook-Toom transforms on integer codes are exact in fp32, so the oracle's fp32
# chains must equal plain integer arithmetic (independent of summation order).
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("m", [2, 4, 6])
def test_input_transform_exact_on_integers(m):
    ct = oracle.cook_toom(m, wi.POINTS[m])
    t = m + 2
    N, C, H, W = 2, 5, 2 * m + 1, m + 3
    x_q = wi.uniform_int8(31 + m, 1, (N, H, W, C))
    L = Layer(N, C, H, W, 4, m, ct["BT32"], ct["G32"], ct["AT32"])
    _, Vf = oracle.input_stage(L, x_q, want_f32=True)
    B4 = np.array([[int(v * 4) for v in row] for row in ct["BT"]], np.int64)   # 4*B^T is integer
    xp = np.pad(x_q.astype(np.int64), ((0, 0), (1, m + 2), (1, m + 2), (0, 0)))
    for n in range(N):
        for th in range(L.TH):
            for tw in range(L.TW):
                tau = (n * L.TH + th) * L.TW + tw
                d = xp[n, th * m: th * m + t, tw * m: tw * m + t, :]
                V16 = np.einsum("ia,abc,jb->ijc", B4, d, B4)
                assert (Vf[:, tau, :].reshape(t, t, C) * 16 == V16).all()


@pytest.mark.parametrize("m", [2, 4])
def test_output_transform_exact_on_integers(m):
    ct = oracle.cook_toom(m, wi.POINTS[m])
    t = m + 2
    N, K, H, W = 1, 3, 2 * m, 2 * m
    L = Layer(N, 4, H, W, K, m, ct["BT32"], ct["G32"], ct["AT32"])
    mq = wi.uniform_int8(41 + m, 1, (t * t, L.T, K))
    _, Yf = oracle.output_stage(L, None, mq, want_f32=True)
    A = np.array([[int(v) for v in row] for row in ct["AT"]], np.int64)
    want = np.einsum("pi,ijtk,qj->tkpq", A, mq.astype(np.int64).reshape(t, t, L.T, K), A)
    assert (Yf == want).all()


# ---------------------------------------------------------------------------
# Exact-rational recomputation of every stage from the previous (quantized)
# stage on tiny layers.
# ---------------------------------------------------------------------------
EPS = Fraction(1, 2 ** 24)


def _frac(a):
    return np.array([Fraction(float(v)) for v in np.asarray(a).flat], dtype=object).reshape(np.shape(a))


def _check_codes(exact_scaled, margin, codes, qmin, qmax, z=0):
    """codes must equal the exactly rounded value unless the exact value is within
    `margin` of a rounding tie.  Returns the number of near-ties."""
    near = 0
    for e, mg, c in zip(exact_scaled.flat, margin.flat, codes.flat):
        fl = e.__floor__()
        frac = e - fl
        dist = abs(frac - Fraction(1, 2))
        if dist <= mg:
            near += 1
            assert abs(int(c) - z - e) <= 1 or int(c) in (qmin, qmax)
            continue
        r = fl + (1 if frac > Fraction(1, 2) else 0)
        want = min(max(r + z, qmin), qmax)
        assert int(c) == want, (float(e), int(c), want)
    return near


@pytest.mark.parametrize("m,flex", [(2, False), (4, False), (6, False), (4, True), (6, True)])
def test_stages_against_exact_rationals(m, flex):
    wl = wi.Workload("tiny", 500 + m + (50 if flex else 0), 1, 3, m + 3, 2 * m + 1, 2, m, flex=flex)
    L, x_q, w_q, bias = build_layer(wl)
    t, T, C, K = L.t, L.T, L.C, L.K
    BT, G, AT = _frac(L.BT), _frac(L.G), _frac(L.AT)
    aBT, aG, aAT = abs(BT), abs(G), abs(AT)
    mul = [Fraction(float(v)) for v in oracle.multipliers(L)]
    Vq, Vf = oracle.input_stage(L, x_q, want_f32=True)
    Uq, Uf = oracle.weight_stage(L, w_q, want_f32=True)
    near = total = 0
    # input stage
    xp = np.pad(x_q.astype(np.int64), ((0, 0), (1, m + 2), (1, m + 2), (0, 0)))
    for tau in range(T):
        th, tw = (tau // L.TW) % L.TH, tau % L.TW
        for c in range(C):
            d = np.array([[Fraction(int(v)) for v in row] for row in xp[0, th * m: th * m + t, tw * m: tw * m + t, c]], dtype=object)
            V = BT.dot(d).dot(BT.T)
            bound = aBT.dot(abs(d)).dot(aBT.T) * (2 * t + 2) * EPS
            got = _frac(Vf[:, tau, c].reshape(t, t))
            assert (abs(got - V) <= bound).all()
            margin = bound * mul[0] + abs(V * mul[0]) * EPS
            near += _check_codes(V * mul[0], margin, Vq[:, tau, c].reshape(t, t), -127, 127)
            total += t * t
    # weight stage
    for k in range(K):
        for c in range(C):
            g = np.array([[Fraction(int(v)) for v in row] for row in w_q[k, :, :, c]], dtype=object)
            U = G.dot(g).dot(G.T)
            bound = aG.dot(abs(g)).dot(aG.T) * 8 * EPS
            got = _frac(Uf[:, k, c].reshape(t, t))
            assert (abs(got - U) <= bound).all()
            margin = bound * mul[1] + abs(U * mul[1]) * EPS
            near += _check_codes(U * mul[1], margin, Uq[:, k, c].reshape(t, t), -127, 127)
            total += t * t
    # Hadamard stage: exact integer definition
    M = oracle.hadamard(L, Vq, Uq)
    want = np.einsum("xtc,xkc->xtk", Vq.astype(np.int64), Uq.astype(np.int64))
    assert (M == want).all()
    assert np.abs(M).max() <= 127 * 127 * C
    mq = oracle.quantize_M(L, M)
    Mf = np.array([Fraction(int(v)) for v in M.flat], dtype=object).reshape(M.shape)
    near += _check_codes(Mf * mul[2], abs(Mf * mul[2]) * EPS, mq, -127, 127)
    total += M.size
    # output stage (right factor first)
    y, Yf = oracle.output_stage(L, M, mq, bias, want_f32=True)
    s_Y = Fraction(float(np.float32(L.q_Y.scale)))
    for tau in range(T):
        th, tw = (tau // L.TW) % L.TH, tau % L.TW
        for k in range(K):
            mm = np.array([Fraction(int(v)) for v in mq[:, tau, k]], dtype=object).reshape(t, t)
            Y = AT.dot(mm).dot(AT.T)
            bound = aAT.dot(abs(mm)).dot(aAT.T) * (2 * t + 2) * EPS
            got = _frac(Yf[tau, k])
            assert (abs(got - Y) <= bound).all()
            bs = Fraction(float(np.float32(float(bias[k]) / float(np.float32(L.q_Y.scale)))))
            for ip in range(m):
                for jp in range(m):
                    h, w = th * m + ip, tw * m + jp
                    if h >= L.H or w >= L.W:
                        continue
                    e = Y[ip, jp] * mul[3] + bs
                    mg = bound[ip, jp] * mul[3] + abs(e) * 2 * EPS
                    near += _check_codes(np.array([e], dtype=object), np.array([mg], dtype=object),
                                         np.array([y[0, h, w, k]]), -127, 127)
                    total += 1
    assert near <= max(3, total // 50), (near, total)


def test_bias_and_float_output_definition():
    wl = wi.Workload("tiny", 77, 1, 4, 5, 5, 3, 2)
    L, x_q, w_q, bias = build_layer(wl, out_dtype=1)
    y, d = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    _, Yf = oracle.output_stage(L, d["M"], d["m_q"], bias, want_f32=True)
    s_M = np.float32(L.q_M.scale)
    tau = 4  # centre tile: (th, tw) = (1, 1)
    want = np.float32(np.float64(Yf[tau, 2, 0, 0]) * np.float64(s_M) + np.float64(bias[2]))
    assert y[0, 2, 2, 2] == want


# ---------------------------------------------------------------------------
# Whole pipeline: sane approximation of the real-valued convolution, error
# growing with the tile size (Section 3.1, "Numerical Error"; Table 1).
# ---------------------------------------------------------------------------
def test_quantized_winograd_tracks_direct_conv_and_degrades_with_m():
    errs = {}
    for m in (2, 4, 6):
        wl = wi.Workload("mid", 900, 2, 32, 12, 12, 16, m)
        L, x_q, w_q, bias = build_layer(wl, out_dtype=1, with_bias=False)
        y = oracle.forward(L, x_q, w_q)
        ref = oracle.direct_conv_i32(x_q, w_q).astype(np.float64) * float(np.float32(L.q_x.scale)) * float(np.float32(L.q_w.scale))
        errs[m] = float(np.sqrt(np.mean((y - ref) ** 2)) / np.sqrt(np.mean(ref ** 2)))
    assert errs[2] < 0.05
    assert errs[2] < errs[4] < errs[6]
    # Table 1: without Winograd-aware training, F4/F6 at 8 bits are unusable
    assert errs[4] > 10 * errs[2]


def test_forward_equals_stagewise_composition_and_pretransformed_weights():
    wl = small(wi.CONFIGS["cfg4"], N=1, C=8, K=8, H=7, W=10)
    L, x_q, w_q, bias = build_layer(wl)
    y, d = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    Vq = oracle.input_stage(L, x_q)
    Uq = oracle.weight_stage(L, w_q)
    M = oracle.hadamard(L, Vq, Uq)
    mq = oracle.quantize_M(L, M)
    y2 = oracle.output_stage(L, M, mq, bias)
    assert (d["V_q"] == Vq).all() and (d["U_q"] == Uq).all() and (d["M"] == M).all() and (d["m_q"] == mq).all()
    assert (y == y2).all()
    y3 = oracle.forward(L, x_q, U_q=Uq, bias=bias)
    assert (y == y3).all()
    assert len(np.unique(y)) > 20


def test_calibrated_scales_fill_the_code_range():
    wl = small(wi.CONFIGS["cfg3"], N=2, C=16, K=16)
    L, x_q, w_q, bias = build_layer(wl)
    _, d = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    for k in ("V_q", "U_q", "m_q"):
        assert np.abs(d[k]).max() == 127
