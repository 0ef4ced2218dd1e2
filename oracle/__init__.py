"""CPU oracle for the Winograd-aware quantized convolution forward pass.

TEST INFRASTRUCTURE ONLY.  This package wraps ``wino_oracle.cpp`` (plain C++,
compiled with g++) through ctypes and numpy.  Nothing in the product package
imports it; only the tests, the smoke check and the benchmark's CPU legs do.
It shares no code with the CUDA library.

Every function follows a passage of the paper:
  cook_toom        Section 3.1 (Cook-Toom construction of G, B^T, A^T)
  input_stage      Eq. 1 / Fig. 2: B^T d B, then Q
  weight_stage     Eq. 1 / Fig. 2: G g G^T, then Q
  hadamard         Sections 1, 5.3: element-wise stage as GEMMs over channels
  quantize_M       Fig. 2: quantized Hadamard output
  output_stage     Eq. 1 / Fig. 2: A^T M A, bias, then Q
  direct_conv_i32  the lossless direct convolution the paper compares against
  winograd_f64     Eq. 1 without any quantizer, in double precision
"""
from __future__ import annotations

import ctypes as ct
import os
import subprocess
from dataclasses import dataclass, field
from fractions import Fraction
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wino_oracle.cpp")
_LIB = os.path.join(_HERE, "libwino_oracle.so")
CXXFLAGS = ["-O2", "-std=c++17", "-fPIC", "-shared", "-fopenmp", "-mfma",
            "-ffp-contract=off", "-fno-fast-math"]


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", *CXXFLAGS, _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class QuantC(ct.Structure):
    _fields_ = [("scale", ct.c_float), ("zero_point", ct.c_int32), ("qmin", ct.c_int32),
                ("qmax", ct.c_int32), ("enabled", ct.c_int32)]


class DescC(ct.Structure):
    _fields_ = [("N", ct.c_int32), ("C", ct.c_int32), ("H", ct.c_int32), ("W", ct.c_int32),
                ("K", ct.c_int32), ("m", ct.c_int32),
                ("BT", ct.c_void_p), ("G", ct.c_void_p), ("AT", ct.c_void_p),
                ("q_x", QuantC), ("q_w", QuantC), ("q_V", QuantC), ("q_U", QuantC),
                ("q_M", QuantC), ("q_Y", QuantC), ("out_dtype", ct.c_int32),
                ("s_w_K", ct.c_void_p), ("s_U_K", ct.c_void_p), ("s_M_K", ct.c_void_p),
                ("s_Y_K", ct.c_void_p)]


@dataclass
class Quant:
    scale: float = 1.0
    zero_point: int = 0
    qmin: int = -127
    qmax: int = 127
    enabled: int = 1

    def c(self) -> QuantC:
        return QuantC(np.float32(self.scale), self.zero_point, self.qmin, self.qmax, self.enabled)


@dataclass
class Layer:
    """Problem statement of one layer: sizes, transform matrices (fp32, as data)
    and the six stage quantizers."""
    N: int
    C: int
    H: int
    W: int
    K: int
    m: int
    BT: np.ndarray
    G: np.ndarray
    AT: np.ndarray
    q_x: Quant = field(default_factory=Quant)
    q_w: Quant = field(default_factory=Quant)
    q_V: Quant = field(default_factory=Quant)
    q_U: Quant = field(default_factory=Quant)
    q_M: Quant = field(default_factory=Quant)
    q_Y: Quant = field(default_factory=Quant)
    out_dtype: int = 0
    # per-output-channel scales (K floats) replacing q_w.scale / q_U.scale / q_M.scale / q_Y.scale
    s_w_K: Optional[np.ndarray] = None
    s_U_K: Optional[np.ndarray] = None
    s_M_K: Optional[np.ndarray] = None
    s_Y_K: Optional[np.ndarray] = None

    @property
    def t(self) -> int:
        return self.m + 2

    @property
    def TH(self) -> int:
        return -(-self.H // self.m)

    @property
    def TW(self) -> int:
        return -(-self.W // self.m)

    @property
    def T(self) -> int:
        return self.N * self.TH * self.TW


_lib = None


def lib() -> ct.CDLL:
    global _lib
    if _lib is None:
        _lib = ct.CDLL(build())
        _lib.orc_quantize.restype = ct.c_int32
        _lib.orc_quantize.argtypes = [ct.c_float, ct.c_float, ct.c_int32, ct.c_int32, ct.c_int32]
        _lib.orc_winograd_f64.restype = ct.c_long
        _lib.orc_direct_f64.restype = ct.c_long
        _lib.orc_num_threads.restype = ct.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ct.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


class _Keep:
    """Holds the descriptor together with the arrays its pointers refer to."""

    def __init__(self, L: Layer):
        self.BT, self.G, self.AT = _f32(L.BT), _f32(L.G), _f32(L.AT)
        t = L.t
        assert self.BT.shape == (t, t) and self.G.shape == (t, 3) and self.AT.shape == (L.m, t)
        self.per_K = []
        for a in (L.s_w_K, L.s_U_K, L.s_M_K, L.s_Y_K):
            if a is not None:
                a = _f32(a)
                assert a.shape == (L.K,) and np.all(a > 0)
            self.per_K.append(a)
        self.d = DescC(L.N, L.C, L.H, L.W, L.K, L.m, _p(self.BT), _p(self.G), _p(self.AT),
                       L.q_x.c(), L.q_w.c(), L.q_V.c(), L.q_U.c(), L.q_M.c(), L.q_Y.c(),
                       L.out_dtype, _p(self.per_K[0]), _p(self.per_K[1]), _p(self.per_K[2]),
                       _p(self.per_K[3]))

    @property
    def ref(self):
        return ct.byref(self.d)


def num_threads() -> int:
    return lib().orc_num_threads()


def set_num_threads(n: int) -> None:
    lib().orc_set_num_threads(ct.c_int(n))


def cook_toom(m: int, points):
    """Section 3.1.  ``points``: m+1 finite points (ints or Fractions).  Returns a
    dict with exact Fraction matrices ('BT','G','AT'), and their correctly
    rounded fp32 / fp64 forms ('BT32', ..., 'BT64', ...)."""
    t = m + 2
    pts = [Fraction(p) for p in points]
    assert len(pts) == t - 1
    pn = np.array([p.numerator for p in pts], dtype=np.int64)
    pd = np.array([p.denominator for p in pts], dtype=np.int64)
    shapes = {"BT": (t, t), "G": (t, 3), "AT": (m, t)}
    num = {k: np.zeros(s, np.int64) for k, s in shapes.items()}
    den = {k: np.zeros(s, np.int64) for k, s in shapes.items()}
    f32 = {k: np.zeros(s, np.float32) for k, s in shapes.items()}
    f64 = {k: np.zeros(s, np.float64) for k, s in shapes.items()}
    rc = lib().orc_cook_toom(ct.c_int(m), _p(pn), _p(pd),
                             _p(num["BT"]), _p(den["BT"]), _p(num["G"]), _p(den["G"]),
                             _p(num["AT"]), _p(den["AT"]),
                             _p(f32["BT"]), _p(f32["G"]), _p(f32["AT"]),
                             _p(f64["BT"]), _p(f64["G"]), _p(f64["AT"]))
    if rc != 0:
        raise ValueError("orc_cook_toom failed")
    out = {}
    for k, s in shapes.items():
        out[k] = np.array([[Fraction(int(num[k][i, j]), int(den[k][i, j])) for j in range(s[1])]
                           for i in range(s[0])], dtype=object)
        out[k + "32"] = f32[k]
        out[k + "64"] = f64[k]
    return out


def quantize(v, mult, z=0, qmin=-127, qmax=127) -> int:
    return int(lib().orc_quantize(ct.c_float(v), ct.c_float(mult), z, qmin, qmax))


def multipliers(L: Layer) -> np.ndarray:
    k = _Keep(L)
    out = np.zeros(5, np.float32)
    lib().orc_multipliers(k.ref, _p(out))
    return out


def input_stage(L: Layer, x_q: np.ndarray, want_f32: bool = False):
    k = _Keep(L)
    x_q = np.ascontiguousarray(x_q, np.int8)
    assert x_q.shape == (L.N, L.H, L.W, L.C)
    shape = (L.t * L.t, L.T, L.C)
    Vq = np.zeros(shape, np.int8)
    Vf = np.zeros(shape, np.float32) if want_f32 else None
    lib().orc_input_stage(k.ref, _p(x_q), _p(Vf), _p(Vq))
    return (Vq, Vf) if want_f32 else Vq


def weight_stage(L: Layer, w_q: np.ndarray, want_f32: bool = False):
    k = _Keep(L)
    w_q = np.ascontiguousarray(w_q, np.int8)
    assert w_q.shape == (L.K, 3, 3, L.C)
    shape = (L.t * L.t, L.K, L.C)
    Uq = np.zeros(shape, np.int8)
    Uf = np.zeros(shape, np.float32) if want_f32 else None
    lib().orc_weight_stage(k.ref, _p(w_q), _p(Uf), _p(Uq))
    return (Uq, Uf) if want_f32 else Uq


def hadamard(L: Layer, V_q: np.ndarray, U_q: np.ndarray) -> np.ndarray:
    k = _Keep(L)
    V_q = np.ascontiguousarray(V_q, np.int8)
    U_q = np.ascontiguousarray(U_q, np.int8)
    assert V_q.shape == (L.t * L.t, L.T, L.C) and U_q.shape == (L.t * L.t, L.K, L.C)
    M = np.zeros((L.t * L.t, L.T, L.K), np.int32)
    lib().orc_hadamard(k.ref, _p(V_q), _p(U_q), _p(M))
    return M


def quantize_M(L: Layer, M: np.ndarray) -> np.ndarray:
    k = _Keep(L)
    M = np.ascontiguousarray(M, np.int32)
    mq = np.zeros(M.shape, np.int8)
    lib().orc_quantize_M(k.ref, _p(M), _p(mq))
    return mq


def output_stage(L: Layer, M, m_q, bias=None, want_f32: bool = False):
    k = _Keep(L)
    M = None if M is None else np.ascontiguousarray(M, np.int32)
    m_q = None if m_q is None else np.ascontiguousarray(m_q, np.int8)
    if L.q_M.enabled:
        assert m_q is not None
    else:
        assert M is not None
    bias = None if bias is None else _f32(bias)
    y = np.zeros((L.N, L.H, L.W, L.K), np.float32 if L.out_dtype == 1 else np.int8)
    Yf = np.zeros((L.T, L.K, L.m, L.m), np.float32) if want_f32 else None
    lib().orc_output_stage(k.ref, _p(M), _p(m_q), _p(bias), _p(Yf), _p(y))
    return (y, Yf) if want_f32 else y


def forward(L: Layer, x_q, w_q=None, U_q=None, bias=None, dumps: bool = False):
    """Whole layer.  Returns y, or (y, dict of stage buffers) when ``dumps``."""
    k = _Keep(L)
    x_q = np.ascontiguousarray(x_q, np.int8)
    assert x_q.shape == (L.N, L.H, L.W, L.C)
    w_q = None if w_q is None else np.ascontiguousarray(w_q, np.int8)
    U_q = None if U_q is None else np.ascontiguousarray(U_q, np.int8)
    bias = None if bias is None else _f32(bias)
    t2 = L.t * L.t
    y = np.zeros((L.N, L.H, L.W, L.K), np.float32 if L.out_dtype == 1 else np.int8)
    d = {}
    if dumps:
        d = {"V_q": np.zeros((t2, L.T, L.C), np.int8), "U_q": np.zeros((t2, L.K, L.C), np.int8),
             "M": np.zeros((t2, L.T, L.K), np.int32), "m_q": np.zeros((t2, L.T, L.K), np.int8)}
    rc = lib().orc_forward(k.ref, _p(x_q), _p(w_q), _p(U_q), _p(bias), _p(y),
                           _p(d.get("V_q")), _p(d.get("U_q")), _p(d.get("M")), _p(d.get("m_q")))
    if rc != 0:
        raise ValueError("orc_forward failed")
    return (y, d) if dumps else y


def direct_conv_i32(x_q, w_q, z_x=0, z_w=0, stride=1) -> np.ndarray:
    x_q = np.ascontiguousarray(x_q, np.int8)
    w_q = np.ascontiguousarray(w_q, np.int8)
    N, H, W, C = x_q.shape
    K = w_q.shape[0]
    assert w_q.shape == (K, 3, 3, C)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    acc = np.zeros((N, Ho, Wo, K), np.int32)
    lib().orc_direct_conv_i32(N, C, H, W, K, stride, _p(x_q), z_x, _p(w_q), z_w, _p(acc))
    return acc


def requantize_acc(acc, s_in: float, q_Y: Quant, bias=None, s_in_K=None, s_Y_K=None) -> np.ndarray:
    """Output quantizer on direct-convolution accumulators; s_in_K (float64, the exact products
    s_x * s_w[k]) and s_Y_K (float32) give per-output-channel scales."""
    acc = np.ascontiguousarray(acc, np.int32)
    K = acc.shape[-1]
    bias = None if bias is None else _f32(bias)
    y = np.zeros(acc.shape, np.int8)
    qc = q_Y.c()
    if s_in_K is not None or s_Y_K is not None:
        s_in_K = None if s_in_K is None else np.ascontiguousarray(s_in_K, np.float64)
        s_Y_K = None if s_Y_K is None else _f32(s_Y_K)
        assert (s_in_K is None or s_in_K.shape == (K,)) and (s_Y_K is None or s_Y_K.shape == (K,))
        lib().orc_requantize_acc_channels(ct.c_long(acc.size), K, _p(acc), ct.c_double(s_in), _p(s_in_K),
                                          _p(bias), ct.byref(qc), _p(s_Y_K), _p(y))
        return y
    lib().orc_requantize_acc(ct.c_long(acc.size), K, _p(acc), ct.c_double(s_in), _p(bias),
                             ct.byref(qc), _p(y))
    return y


def winograd_f64(x, w, m, BT, G, AT, pad=1):
    x = np.ascontiguousarray(x, np.float64)
    w = np.ascontiguousarray(w, np.float64)
    BT, G, AT = (np.ascontiguousarray(a, np.float64) for a in (BT, G, AT))
    N, H, W, C = x.shape
    K = w.shape[0]
    Ho, Wo = H + 2 * pad - 2, W + 2 * pad - 2
    y = np.zeros((N, Ho, Wo, K), np.float64)
    mults = lib().orc_winograd_f64(N, C, H, W, K, m, pad, _p(BT), _p(G), _p(AT), _p(x), _p(w), _p(y))
    return y, int(mults)


def direct_f64(x, w, pad=1):
    x = np.ascontiguousarray(x, np.float64)
    w = np.ascontiguousarray(w, np.float64)
    N, H, W, C = x.shape
    K = w.shape[0]
    Ho, Wo = H + 2 * pad - 2, W + 2 * pad - 2
    y = np.zeros((N, Ho, Wo, K), np.float64)
    mults = lib().orc_direct_f64(N, C, H, W, K, pad, _p(x), _p(w), _p(y))
    return y, int(mults)
