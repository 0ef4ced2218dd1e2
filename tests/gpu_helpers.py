"""Helpers for the GPU parity tests: run a layer through the C ABI (via the thin
binding) and hand back numpy arrays."""
from __future__ import annotations

import numpy as np
import torch

from paper_2002_10711_b200 import binding
from paper_2002_10711_b200.layer import WinogradConv


def gpu_run(L, x_q, w_q, bias, path=binding.PATH_AUTO, dumps=False):
    plan = binding.Plan.from_layer(L, path=path)
    conv = WinogradConv(plan)
    conv.load_weights(w_q, bias)
    x = torch.from_numpy(np.ascontiguousarray(x_q)).cuda()
    y = conv.forward(x)
    st = plan.last_status()
    assert st == 0, binding.strerror(st)
    out = {"y": y.cpu().numpy(), "U_q": conv.Uq.cpu().numpy().reshape(L.t * L.t, L.K, L.C),
           "path": plan.path, "launches": plan.launch_count}
    if plan.path in (binding.PATH_SMALLC, binding.PATH_FUSED_F2):
        # single-kernel paths: a second pass that also writes the int32 Hadamard sums
        M = torch.full((L.t * L.t, plan.T, L.K), -1, dtype=torch.int32, device="cuda")
        y2 = conv.empty_output()
        plan.debug_forward_accumulators(x, conv.Uq, conv.bias, y2, M, M.numel() * 4)
        assert plan.last_status() == 0
        assert torch.equal(y2, y)
        out["M"] = M.cpu().numpy()
    if dumps:
        out["V_q"] = conv.dump(binding.STAGE_VQ).cpu().numpy()
        out["M"] = conv.dump(binding.STAGE_M_I32).cpu().numpy()
        if L.q_M.enabled:
            out["m_q"] = conv.dump(binding.STAGE_MQ).cpu().numpy()
        assert plan.last_status() == 0
    return out
