"""ctypes binding of the C ABI in include/wino.h.

Argument marshalling only: every step of the layer runs in the CUDA library.
PyTorch is used for device memory and streams.  If the shared library is
missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes as ct
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwino_b200.so")

WINO_OK = 0
ERR_INVALID, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
PATH_AUTO, PATH_STAGED_TC, PATH_STAGED_DP4A, PATH_SMALLC, PATH_STAGED_TC_PTR = 0, 1, 2, 3, 4
PATH_FUSED_F2 = 5
PATH_STAGED_TC_MMA = 6
PATH_FUSED_LAYER = 7
STAGE_VQ, STAGE_M_I32, STAGE_MQ = 0, 1, 2
STATIC_SCRATCH_BYTES = 20 * 1024 * 1024

EXPORTS = [
    "wino_plan", "wino_weight_bytes", "wino_workspace_bytes", "wino_plan_path",
    "wino_plan_force_path", "wino_plan_set_channel_scales", "wino_plan_multipliers",
    "wino_transform_weights", "wino_transform_weights_channel_stats",
    "wino_conv_forward", "wino_conv_forward_static", "wino_calibrate_forward",
    "wino_direct_conv_forward", "wino_direct_last_status", "wino_last_status", "wino_debug_dump_stage",
    "wino_debug_forward_accumulators", "wino_debug_run_stages", "wino_debug_mma_probe",
    "wino_debug_wait_probe", "wino_debug_once_per_device", "wino_launch_count", "wino_destroy",
    "wino_strerror",
]


class QuantC(ct.Structure):
    _fields_ = [("scale", ct.c_float), ("zero_point", ct.c_int32), ("qmin", ct.c_int32),
                ("qmax", ct.c_int32), ("enabled", ct.c_int32)]


class DescC(ct.Structure):
    _fields_ = [("N", ct.c_int32), ("C", ct.c_int32), ("H", ct.c_int32), ("W", ct.c_int32),
                ("K", ct.c_int32), ("m", ct.c_int32),
                ("BT", ct.c_void_p), ("G", ct.c_void_p), ("AT", ct.c_void_p),
                ("transforms_exact", ct.c_int32),
                ("q_x", QuantC), ("q_w", QuantC), ("q_V", QuantC), ("q_U", QuantC),
                ("q_M", QuantC), ("q_Y", QuantC), ("out_dtype", ct.c_int32)]


class DirectDescC(ct.Structure):
    _fields_ = [("N", ct.c_int32), ("C", ct.c_int32), ("H", ct.c_int32), ("W", ct.c_int32),
                ("K", ct.c_int32), ("stride", ct.c_int32),
                ("q_x", QuantC), ("q_w", QuantC), ("q_Y", QuantC), ("out_dtype", ct.c_int32),
                ("s_w_K_dev", ct.c_void_p), ("s_Y_K_dev", ct.c_void_p)]


class WinoError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


def _load() -> ct.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2002_10711_b200.build` "
            "(there is no CPU fallback)")
    lib = ct.CDLL(LIB_PATH)
    vp, i32, sz = ct.c_void_p, ct.c_int, ct.c_size_t
    lib.wino_plan.argtypes = [ct.POINTER(DescC), ct.POINTER(vp)]
    lib.wino_weight_bytes.argtypes = [vp]
    lib.wino_weight_bytes.restype = sz
    lib.wino_workspace_bytes.argtypes = [vp]
    lib.wino_workspace_bytes.restype = sz
    lib.wino_plan_path.argtypes = [vp]
    lib.wino_plan_force_path.argtypes = [vp, i32]
    lib.wino_plan_set_channel_scales.argtypes = [vp, vp, vp, vp, vp]
    lib.wino_plan_multipliers.argtypes = [vp, vp]
    lib.wino_transform_weights.argtypes = [vp, vp, vp, vp, vp]
    lib.wino_transform_weights_channel_stats.argtypes = [vp, vp, vp, vp, vp]
    lib.wino_conv_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.wino_conv_forward_static.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.wino_calibrate_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.wino_debug_run_stages.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.wino_direct_conv_forward.argtypes = [ct.POINTER(DirectDescC), vp, vp, vp, vp, vp]
    lib.wino_direct_last_status.argtypes = [vp]
    lib.wino_debug_mma_probe.argtypes = [vp, i32, vp]
    lib.wino_last_status.argtypes = [vp, vp]
    lib.wino_debug_dump_stage.argtypes = [vp, i32, vp, sz]
    lib.wino_launch_count.argtypes = [vp]
    lib.wino_launch_count.restype = ct.c_long
    lib.wino_debug_forward_accumulators.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.wino_debug_wait_probe.argtypes = [vp, ct.c_longlong, vp]
    lib.wino_debug_once_per_device.argtypes = [i32]
    lib.wino_destroy.argtypes = [vp]
    lib.wino_destroy.restype = None
    lib.wino_strerror.argtypes = [i32]
    lib.wino_strerror.restype = ct.c_char_p
    return lib


_lib = _load()


def strerror(code: int) -> str:
    return _lib.wino_strerror(code).decode()


def _check(rc: int, what: str) -> None:
    if rc != WINO_OK:
        raise WinoError(rc, what)


def _quant(q) -> QuantC:
    """q: object with scale, zero_point, qmin, qmax, enabled (or a dict)."""
    g = (lambda k, d: q.get(k, d)) if isinstance(q, dict) else (lambda k, d: getattr(q, k, d))
    return QuantC(np.float32(g("scale", 1.0)), int(g("zero_point", 0)), int(g("qmin", -127)),
                  int(g("qmax", 127)), int(g("enabled", 1)))


def _dptr(t):
    """Device (or host) address of a torch tensor / raw int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return ct.c_void_p(t)
    return ct.c_void_p(t.data_ptr())


def _stream_handle(stream) -> ct.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ct.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def debug_once_per_device(device: int) -> int:
    return _lib.wino_debug_once_per_device(device)


def direct_last_status(stream=None) -> int:
    """wino_direct_last_status: status word of the plan-less direct convolutions (read and cleared)."""
    return int(_lib.wino_direct_last_status(_stream_handle(stream)))


def direct_conv_forward(N, C, H, W, K, stride, q_x, q_w, q_Y, x_dev, w_dev, bias_dev, y_dev,
                        out_dtype=0, stream=None, s_w_K_dev=None, s_Y_K_dev=None) -> None:
    """wino_direct_conv_forward: direct int8 3x3 convolution, stride 1 or 2; s_w_K_dev and
    s_Y_K_dev: optional per-output-channel scales (float32 tensors of K elements on the device)."""
    d = DirectDescC(N, C, H, W, K, stride, _quant(q_x), _quant(q_w), _quant(q_Y), out_dtype,
                    None if s_w_K_dev is None else s_w_K_dev.data_ptr(),
                    None if s_Y_K_dev is None else s_Y_K_dev.data_ptr())
    _check(_lib.wino_direct_conv_forward(ct.byref(d), _dptr(x_dev), _dptr(w_dev), _dptr(bias_dev),
                                         _dptr(y_dev), _stream_handle(stream)),
           "wino_direct_conv_forward")


class Plan:
    """Owns a wino_plan_t*.  Mirrors the C entry points one to one."""

    def __init__(self, N, C, H, W, K, m, BT, G, AT, q_x, q_w, q_V, q_U, q_M, q_Y,
                 out_dtype=0, transforms_exact=0, path=PATH_AUTO):
        t = m + 2
        self._BT = np.ascontiguousarray(BT, np.float32)
        self._G = np.ascontiguousarray(G, np.float32)
        self._AT = np.ascontiguousarray(AT, np.float32)
        if m in (2, 4, 6) and (self._BT.shape != (t, t) or self._G.shape != (t, 3) or self._AT.shape != (m, t)):
            raise ValueError("matrix shapes must be BT[t,t], G[t,3], AT[m,t]")
        self.desc = DescC(N, C, H, W, K, m, self._BT.ctypes.data, self._G.ctypes.data,
                          self._AT.ctypes.data, transforms_exact, _quant(q_x), _quant(q_w),
                          _quant(q_V), _quant(q_U), _quant(q_M), _quant(q_Y), out_dtype)
        self._h = ct.c_void_p()
        _check(_lib.wino_plan(ct.byref(self.desc), ct.byref(self._h)), "wino_plan")
        self.N, self.C, self.H, self.W, self.K, self.m, self.t = N, C, H, W, K, m, t
        self.TH, self.TW = -(-H // m), -(-W // m)
        self.T = N * self.TH * self.TW
        self.out_dtype = out_dtype
        if path != PATH_AUTO:
            self.force_path(path)

    @classmethod
    def from_layer(cls, L, **kw):
        """L: any object with fields N,C,H,W,K,m,BT,G,AT,q_x..q_Y,out_dtype and, optionally,
        per-output-channel scales s_w_K, s_U_K, s_M_K, s_Y_K."""
        plan = cls(L.N, L.C, L.H, L.W, L.K, L.m, L.BT, L.G, L.AT, L.q_x, L.q_w, L.q_V, L.q_U,
                   L.q_M, L.q_Y, out_dtype=L.out_dtype, **kw)
        per_K = [getattr(L, n, None) for n in ("s_w_K", "s_U_K", "s_M_K", "s_Y_K")]
        if any(a is not None for a in per_K):
            plan.set_channel_scales(*per_K)
        return plan

    def __del__(self):
        h = getattr(self, "_h", None)
        if h is not None and h.value and _lib is not None:
            _lib.wino_destroy(h)
            self._h = ct.c_void_p()

    # --- queries ---
    @property
    def weight_bytes(self) -> int:
        return _lib.wino_weight_bytes(self._h)

    @property
    def workspace_bytes(self) -> int:
        return _lib.wino_workspace_bytes(self._h)

    @property
    def path(self) -> int:
        return _lib.wino_plan_path(self._h)

    def force_path(self, path: int) -> None:
        _check(_lib.wino_plan_force_path(self._h, path), "wino_plan_force_path")

    def set_channel_scales(self, s_w_K=None, s_U_K=None, s_M_K=None, s_Y_K=None) -> None:
        """Per-output-channel scales (K floats each; None keeps the per-layer scale)."""
        keep = [None if a is None else np.ascontiguousarray(a, np.float32) for a in (s_w_K, s_U_K, s_M_K, s_Y_K)]
        for a in keep:
            if a is not None and a.shape != (self.K,):
                raise ValueError("channel scales must have shape (K,)")
        _check(_lib.wino_plan_set_channel_scales(
            self._h, *[None if a is None else a.ctypes.data for a in keep]), "wino_plan_set_channel_scales")

    def multipliers(self) -> np.ndarray:
        out = np.zeros(5, np.float32)
        _check(_lib.wino_plan_multipliers(self._h, out.ctypes.data), "wino_plan_multipliers")
        return out

    @property
    def launch_count(self) -> int:
        return _lib.wino_launch_count(self._h)

    # --- device entry points ---
    def transform_weights(self, w_dev, Uq_dev, absmax_dev=None, stream=None) -> None:
        _check(_lib.wino_transform_weights(self._h, _dptr(w_dev), _dptr(Uq_dev), _dptr(absmax_dev),
                                           _stream_handle(stream)), "wino_transform_weights")

    def transform_weights_channel_stats(self, w_dev, Uq_dev, absmax_K_dev, stream=None) -> None:
        _check(_lib.wino_transform_weights_channel_stats(
            self._h, _dptr(w_dev), _dptr(Uq_dev), _dptr(absmax_K_dev), _stream_handle(stream)),
            "wino_transform_weights_channel_stats")

    def conv_forward(self, x_dev, Uq_dev, bias_dev, y_dev, workspace_dev, stream=None) -> None:
        _check(_lib.wino_conv_forward(self._h, _dptr(x_dev), _dptr(Uq_dev), _dptr(bias_dev),
                                      _dptr(y_dev), _dptr(workspace_dev), _stream_handle(stream)),
               "wino_conv_forward")

    def conv_forward_static(self, x_dev, Uq_dev, bias_dev, y_dev, stream=None) -> None:
        """wino_conv_forward_static: no workspace argument; the library's built-in static
        scratch (STATIC_SCRATCH_BYTES at most) is used, and nothing is allocated."""
        _check(_lib.wino_conv_forward_static(self._h, _dptr(x_dev), _dptr(Uq_dev), _dptr(bias_dev),
                                             _dptr(y_dev), _stream_handle(stream)),
               "wino_conv_forward_static")

    def debug_run_stages(self, stage_mask, x_dev, Uq_dev, bias_dev, y_dev, workspace_dev,
                         stream=None) -> None:
        _check(_lib.wino_debug_run_stages(self._h, stage_mask, _dptr(x_dev), _dptr(Uq_dev),
                                          _dptr(bias_dev), _dptr(y_dev), _dptr(workspace_dev),
                                          _stream_handle(stream)), "wino_debug_run_stages")

    def debug_mma_probe(self, iters: int, stream=None) -> None:
        _check(_lib.wino_debug_mma_probe(self._h, iters, _stream_handle(stream)),
               "wino_debug_mma_probe")

    def calibrate_forward(self, x_dev, Uq_dev, bias_dev, y_dev, workspace_dev, absmax4_dev,
                          stream=None) -> None:
        _check(_lib.wino_calibrate_forward(self._h, _dptr(x_dev), _dptr(Uq_dev), _dptr(bias_dev),
                                           _dptr(y_dev), _dptr(workspace_dev), _dptr(absmax4_dev),
                                           _stream_handle(stream)), "wino_calibrate_forward")

    def debug_wait_probe(self, limit_cycles: int, stream=None) -> None:
        _check(_lib.wino_debug_wait_probe(self._h, limit_cycles, _stream_handle(stream)),
               "wino_debug_wait_probe")

    def debug_forward_accumulators(self, x_dev, Uq_dev, bias_dev, y_dev, M_dev, nbytes: int,
                                   stream=None) -> None:
        _check(_lib.wino_debug_forward_accumulators(self._h, _dptr(x_dev), _dptr(Uq_dev),
                                                    _dptr(bias_dev), _dptr(y_dev), _dptr(M_dev),
                                                    nbytes, _stream_handle(stream)),
               "wino_debug_forward_accumulators")

    def last_status(self, stream=None) -> int:
        """Synchronizes the stream; returns the device status word and clears it."""
        return _lib.wino_last_status(self._h, _stream_handle(stream))

    def debug_dump_stage(self, stage: int, dst_dev, nbytes: int) -> None:
        _check(_lib.wino_debug_dump_stage(self._h, stage, _dptr(dst_dev), nbytes),
               "wino_debug_dump_stage")
