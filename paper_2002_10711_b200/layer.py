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
