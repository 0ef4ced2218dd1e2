"""One-shot max-abs calibration of the four inner stage scales through the oracle.

TEST INFRASTRUCTURE (part of the CPU oracle).  The paper sets every stage's
range from moving averages over training data (Table 1 caption, "warmup of all
the moving averages"); with no data here, each scale is the max-abs of its
stage on the seeded batch, taken stage by stage on the already-quantized
previous stage, s = max|real value| / 127 rounded once to fp32 (per-layer
symmetric quantization, Section 5.1).  The resulting scales are plain inputs to
both the oracle and the CUDA library.
"""
from __future__ import annotations

import copy

import numpy as np

from . import Layer, hadamard, input_stage, output_stage, quantize_M, weight_stage


def _scale(maxabs_real: float) -> float:
    return float(np.float32(maxabs_real / 127.0)) if maxabs_real > 0 else 1.0


def calibrate(L: Layer, x_q, w_q, bias=None) -> Layer:
    """Returns a copy of L with q_V, q_U, q_M, q_Y scales filled in."""
    L = copy.deepcopy(L)
    _, Vf = input_stage(L, x_q, want_f32=True)
    L.q_V.scale = _scale(float(np.max(np.abs(Vf))) * float(np.float32(L.q_x.scale)))
    _, Uf = weight_stage(L, w_q, want_f32=True)
    L.q_U.scale = _scale(float(np.max(np.abs(Uf))) * float(np.float32(L.q_w.scale)))
    Vq = input_stage(L, x_q)
    Uq = weight_stage(L, w_q)
    M = hadamard(L, Vq, Uq)
    if L.q_M.enabled:
        sUV = float(np.float32(L.q_U.scale)) * float(np.float32(L.q_V.scale))
        L.q_M.scale = _scale(float(np.max(np.abs(M))) * sUV)
        mq = quantize_M(L, M)
    else:
        mq = None
    Lf = copy.deepcopy(L)
    Lf.out_dtype = 1
    yf = output_stage(Lf, M, mq, bias)
    L.q_Y.scale = _scale(float(np.max(np.abs(yf))))
    return L


def calibrate_per_channel(L: Layer, x_q, w_q, bias=None, output_per_channel: bool = False) -> Layer:
    """Per-output-channel variant (Section 7): L.s_w_K must be set (the scales the filters in
    w_q were quantized with); fills q_V, s_U_K (max-abs of each transformed filter), s_M_K
    (max-abs of each channel's Hadamard sums) and q_Y (one scale: the next layer sums over
    these channels), or s_Y_K when ``output_per_channel``."""
    assert L.s_w_K is not None
    L = copy.deepcopy(L)
    L.s_U_K = None
    L.s_M_K = None
    L.s_Y_K = None
    s_w = np.asarray(L.s_w_K, np.float32).astype(np.float64)
    _, Vf = input_stage(L, x_q, want_f32=True)
    L.q_V.scale = _scale(float(np.max(np.abs(Vf))) * float(np.float32(L.q_x.scale)))
    _, Uf = weight_stage(L, w_q, want_f32=True)                  # [t*t][K][C], code units
    u_max = np.max(np.abs(Uf.astype(np.float64)), axis=(0, 2)) * s_w
    L.s_U_K = np.array([_scale(v) for v in u_max], np.float32)
    Vq = input_stage(L, x_q)
    Uq = weight_stage(L, w_q)
    M = hadamard(L, Vq, Uq)
    sUV = L.s_U_K.astype(np.float64) * float(np.float32(L.q_V.scale))
    if L.q_M.enabled:
        L.s_M_K = np.array([_scale(v) for v in np.abs(M).max(axis=(0, 1)) * sUV], np.float32)
        mq = quantize_M(L, M)
    else:
        mq = None
    Lf = copy.deepcopy(L)
    Lf.out_dtype = 1
    yf = output_stage(Lf, M, mq, bias)
    if output_per_channel:
        L.s_Y_K = np.array([_scale(v) for v in np.abs(yf).max(axis=(0, 1, 2))], np.float32)
    else:
        L.q_Y.scale = _scale(float(np.max(np.abs(yf))))
    return L
