"""Convenience wrapper: one Winograd-aware quantized conv layer on the GPU.

Holds a Plan plus the device buffers it needs (transformed weights, workspace).
All arithmetic happens in the CUDA library; torch only owns memory and streams.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding
from .binding import Plan


class WinogradConv:
    def __init__(self, plan: Plan, device="cuda:0"):
        self.plan = plan
        self.device = torch.device(device)
        self.Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device=self.device)
        self.ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device=self.device)
        self.bias = None

    def load_weights(self, w_q, bias=None, absmax=None) -> None:
        """w_q: int8 [K,3,3,C] (numpy or torch); runs the weight transform."""
        w = torch.as_tensor(np.ascontiguousarray(w_q) if isinstance(w_q, np.ndarray) else w_q)
        w = w.to(self.device, torch.int8).contiguous()
        self.plan.transform_weights(w, self.Uq, absmax)
        self.bias = None if bias is None else torch.as_tensor(bias).to(self.device, torch.float32).contiguous()
        torch.cuda.current_stream().synchronize()  # w may be freed after return

    def empty_output(self) -> torch.Tensor:
        p = self.plan
        dt = torch.float32 if p.out_dtype == 1 else torch.int8
        return torch.empty((p.N, p.H, p.W, p.K), dtype=dt, device=self.device)

    def forward(self, x_dev: torch.Tensor, y_dev: torch.Tensor | None = None) -> torch.Tensor:
        """x_dev: int8 [N,H,W,C] on the device."""
        if y_dev is None:
            y_dev = self.empty_output()
        self.plan.conv_forward(x_dev, self.Uq, self.bias, y_dev, self.ws)
        return y_dev

    def dump(self, stage: int) -> torch.Tensor:
        p = self.plan
        t2 = p.t * p.t
        if stage == binding.STAGE_VQ:
            out = torch.empty((t2, p.T, p.C), dtype=torch.int8, device=self.device)
        elif stage == binding.STAGE_MQ:
            out = torch.empty((t2, p.T, p.K), dtype=torch.int8, device=self.device)
        else:
            out = torch.empty((t2, p.T, p.K), dtype=torch.int32, device=self.device)
        p.debug_dump_stage(stage, out, out.numel() * out.element_size())
        return out


def calibrate(make_plan, x_q, w_q, bias, s_x: float, s_w: float, device="cuda:0"):
    """One-shot max-abs calibration of the four inner stage scales on the GPU
    (stand-in for the paper's moving-average range observers, Table 1 caption).

    make_plan(s_V, s_U, s_M, s_Y) -> Plan builds a plan with the given scales.
    Each scale is max|real value of the stage| / 127, rounded once to fp32, taken
    stage by stage on the already-quantized previous stage.  Returns
    (s_V, s_U, s_M, s_Y) as Python floats."""
    dev = torch.device(device)
    x = torch.as_tensor(np.ascontiguousarray(x_q)).to(dev, torch.int8)
    w = torch.as_tensor(np.ascontiguousarray(w_q)).to(dev, torch.int8)
    b = None if bias is None else torch.as_tensor(bias).to(dev, torch.float32)
    f32 = lambda v: float(np.float32(v))
    scale = lambda mx: f32(mx / 127.0) if mx > 0 else 1.0

    def run(s_V, s_U, s_M, s_Y):
        plan = make_plan(s_V, s_U, s_M, s_Y)
        Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device=dev)
        ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
        am = torch.zeros(8, dtype=torch.int32, device=dev)
        plan.transform_weights(w, Uq, am[4:])
        plan.calibrate_forward(x, Uq, b, None, ws, am)
        st = plan.last_status()
        if st != 0:
            raise binding.WinoError(st, "calibrate")
        return am.cpu().numpy().view(np.float32)

    enabled = bool(make_plan(1.0, 1.0, 1.0, 1.0).desc.q_M.enabled)
    a = run(1.0, 1.0, 1.0, 1.0)
    s_V = scale(float(a[0]) * f32(s_x))
    s_U = scale(float(a[4]) * f32(s_w))
    a = run(s_V, s_U, 1.0, 1.0)
    s_M = scale(float(a[1]) * (s_U * s_V)) if enabled else 1.0
    a = run(s_V, s_U, s_M, 1.0)
    s_Y = scale(float(a[3]))
    return s_V, s_U, s_M, s_Y


def calibrate_per_channel(make_plan, x_q, w_q, bias, s_x: float, s_w_K, output_per_channel: bool = False,
                          device="cuda:0"):
    """Max-abs calibration with per-output-channel scales (Section 7) on the GPU.

    make_plan(s_V, s_U, s_M, s_Y, out_dtype) -> Plan builds a plan with the given per-layer
    scales and output type; s_w_K are the scales the filters in w_q were quantized with.
    Stage by stage on the already-quantized previous stage: s_V (one scale, from the
    calibration pass), s_U[k] from the weight transform's per-filter statistic, s_M[k] from
    the int32 Hadamard sums (dumped and reduced with torch: plumbing, not the layer's path),
    then the output: one s_Y (a layer inside a network: the next layer sums over these
    channels) or s_Y[k].  Returns (s_V, s_U_K, s_M_K or None, s_Y or s_Y_K)."""
    dev = torch.device(device)
    x = torch.as_tensor(np.ascontiguousarray(x_q)).to(dev, torch.int8)
    w = torch.as_tensor(np.ascontiguousarray(w_q)).to(dev, torch.int8)
    b = None if bias is None else torch.as_tensor(bias).to(dev, torch.float32)
    s_w_K = np.ascontiguousarray(s_w_K, np.float32)
    f32 = lambda v: float(np.float32(v))
    scale = lambda mx: f32(mx / 127.0) if mx > 0 else 1.0
    scales = lambda arr: np.array([scale(float(v)) for v in arr], np.float32)

    def check(plan):
        st = plan.last_status()
        if st != 0:
            raise binding.WinoError(st, "calibrate_per_channel")

    # input side and the transformed filters
    plan = make_plan(1.0, 1.0, 1.0, 1.0, 0)
    K = plan.K
    plan.set_channel_scales(s_w_K, None, None, None)
    Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device=dev)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    am = torch.zeros(4, dtype=torch.int32, device=dev)
    amK = torch.zeros(K, dtype=torch.int32, device=dev)
    plan.transform_weights_channel_stats(w, Uq, amK)
    plan.calibrate_forward(x, Uq, b, None, ws, am)
    check(plan)
    s_V = scale(float(am.cpu().numpy().view(np.float32)[0]) * f32(s_x))
    u_max = amK.cpu().numpy().view(np.float32).astype(np.float64) * s_w_K.astype(np.float64)
    s_U_K = scales(u_max)
    enabled = bool(plan.desc.q_M.enabled)

    # Hadamard sums under the final V and U scales
    conv = WinogradConv(make_plan(s_V, 1.0, 1.0, 1.0, 0), device=device)
    conv.plan.set_channel_scales(s_w_K, s_U_K, None, None)
    conv.load_weights(w, b)
    conv.forward(x)
    M = conv.dump(binding.STAGE_M_I32)
    check(conv.plan)
    m_max = M.abs().amax(dim=(0, 1)).cpu().numpy().astype(np.float64)
    s_M_K = scales(m_max * (s_U_K.astype(np.float64) * s_V)) if enabled else None

    # the real-valued output under the final inner scales
    conv = WinogradConv(make_plan(s_V, 1.0, 1.0, 1.0, 1), device=device)
    conv.plan.set_channel_scales(s_w_K, s_U_K, s_M_K, None)
    conv.load_weights(w, b)
    y = conv.forward(x)
    check(conv.plan)
    if output_per_channel:
        return s_V, s_U_K, s_M_K, scales(y.abs().amax(dim=(0, 1, 2)).cpu().numpy())
    return s_V, s_U_K, s_M_K, scale(float(y.abs().max()))
