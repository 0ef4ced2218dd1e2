"""Shared test helpers: build a layer statement (sizes, matrices, scales) for a
seeded workload.  Matrices and calibrated scales come from the oracle and are
handed to both sides as data."""
from __future__ import annotations

import copy

import numpy as np

import oracle
import wino_inputs as wi
from oracle import Layer, Quant
from oracle.calibrate import calibrate


def matrices(m: int, flex_seed: int | None = None):
    ct = oracle.cook_toom(m, wi.POINTS[m])
    BT, G, AT = ct["BT32"], ct["G32"], ct["AT32"]
    if flex_seed is not None:
        BT = wi.flex_perturb(BT, flex_seed, wi.S_BT)
        G = wi.flex_perturb(G, flex_seed, wi.S_G)
        AT = wi.flex_perturb(AT, flex_seed, wi.S_AT)
    return BT, G, AT


def build_layer(wl: wi.Workload, N: int | None = None, q_M: bool = True, out_dtype: int = 0,
                with_bias: bool = True, relu: bool = False):
    """Returns (Layer, x_q, w_q, bias) with every scale fixed."""
    x_q, s_x, w_q, s_w, bias = wi.make_tensors(wl, N=N, with_bias=with_bias)
    BT, G, AT = matrices(wl.m, wl.seed if wl.flex else None)
    L = Layer(N=x_q.shape[0], C=wl.C, H=wl.H, W=wl.W, K=wl.K, m=wl.m, BT=BT, G=G, AT=AT,
              out_dtype=out_dtype)
    L.q_x = Quant(scale=float(s_x))
    L.q_w = Quant(scale=float(s_w))
    L.q_M = Quant(enabled=1 if q_M else 0)
    if relu:
        L.q_Y = Quant(qmin=0)
    if wl.fixed_scales is not None:
        for q in (L.q_V, L.q_U, L.q_M, L.q_Y):
            q.scale = float(np.float32(wl.fixed_scales))
    else:
        L = calibrate(L, x_q, w_q, bias)
    return L, x_q, w_q, bias


def per_channel(L: Layer, seed: int, spread: float = 2.0) -> Layer:
    """Copy of L whose weight, transformed-weight, Hadamard-sum and output scales vary per output channel
    (the per-layer scale times a seeded factor in [1/spread, spread])."""
    f_w, f_U, f_M, f_Y = wi.channel_factors(seed, L.K, spread)
    P = copy.deepcopy(L)
    P.s_w_K = (np.float32(L.q_w.scale) * f_w).astype(np.float32)
    P.s_U_K = (np.float32(L.q_U.scale) * f_U).astype(np.float32)
    P.s_M_K = (np.float32(L.q_M.scale) * f_M).astype(np.float32) if L.q_M.enabled else None
    P.s_Y_K = (np.float32(L.q_Y.scale) * f_Y).astype(np.float32)
    return P


def small(wl: wi.Workload, **kw) -> wi.Workload:
    d = copy.copy(wl.__dict__)
    d.update(kw)
    return wi.Workload(**d)
