"""No kernel may write outside its buffers: inputs, weights, workspace and output
are carved out of one arena with guard bands between them, and the guard bytes
must be untouched after a forward pass (ragged tile counts, clipped TMA boxes,
partial blocks), on every path the shape supports."""
import numpy as np
import pytest

import oracle
import wino_inputs as wi
from helpers import build_layer

pytestmark = pytest.mark.gpu

GUARD = 8192
FILL = 0xA5


def _carve(arena, sizes):
    import torch
    views, off = [], GUARD
    for n in sizes:
        views.append(arena[off: off + n])
        off += (n + 1023) // 1024 * 1024 + GUARD
    return views


@pytest.mark.parametrize("shape,m", [((3, 128, 7, 9, 192), 4), ((2, 64, 13, 5, 64), 6), ((5, 64, 9, 11, 64), 2),
                                     ((1, 256, 6, 6, 256), 6), ((2, 48, 10, 7, 80), 4), ((3, 16, 5, 9, 24), 2)])
def test_guard_bands_stay_intact(shape, m):
    import torch
    from paper_2002_10711_b200 import binding
    N, C, H, W, K = shape
    wl = wi.Workload("g", 4100 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    y_ref = oracle.forward(L, x_q, w_q, bias=bias)
    auto = binding.Plan.from_layer(L).path
    paths = {auto, binding.PATH_STAGED_DP4A}
    if C % 16 == 0 and K % 16 == 0:
        paths |= {binding.PATH_STAGED_TC, binding.PATH_STAGED_TC_PTR}
    for path in sorted(paths):
        plan = binding.Plan.from_layer(L, path=path)
        sizes = [x_q.size, w_q.size, plan.weight_bytes, max(plan.workspace_bytes, 16), y_ref.size, K * 4]
        total = GUARD + sum((n + 1023) // 1024 * 1024 + GUARD for n in sizes)
        arena = torch.full((total,), FILL, dtype=torch.uint8, device="cuda")
        xb, wb, ub, wsb, yb, bb = _carve(arena, sizes)
        xb.copy_(torch.from_numpy(x_q.reshape(-1).view(np.uint8)))
        wb.copy_(torch.from_numpy(w_q.reshape(-1).view(np.uint8)))
        bb.copy_(torch.from_numpy(bias.view(np.uint8)))
        plan.transform_weights(wb, ub)
        plan.conv_forward(xb, ub, bb, yb, wsb)
        assert plan.last_status() == 0
        host = arena.cpu().numpy()
        got = yb.cpu().numpy().view(np.int8).reshape(y_ref.shape)
        assert (got == y_ref).all(), path
        mask = np.ones(total, bool)
        off = GUARD
        for n in sizes:
            mask[off: off + n] = False
            off += (n + 1023) // 1024 * 1024 + GUARD
        assert (host[mask] == FILL).all(), f"path {path}: a guard byte was overwritten"


@pytest.mark.parametrize("shape,m", [((8, 256, 8, 8, 256), 4), ((3, 128, 7, 9, 128), 2), ((2, 64, 9, 9, 64), 6)])
def test_buffers_aligned_to_sixteen_bytes_only(shape, m):
    # the header promises nothing beyond 16-byte alignment of the device pointers: every buffer
    # sits 16 bytes past a 1024-byte boundary here
    import torch
    from paper_2002_10711_b200 import binding
    N, C, H, W, K = shape
    wl = wi.Workload("a16", 4200 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    y_ref = oracle.forward(L, x_q, w_q, bias=bias)
    for path in (binding.PATH_STAGED_TC, binding.PATH_STAGED_TC_PTR, binding.PATH_STAGED_DP4A):
        plan = binding.Plan.from_layer(L, path=path)
        sizes = [x_q.size, w_q.size, plan.weight_bytes, max(plan.workspace_bytes, 16), y_ref.size, K * 4]
        bufs = []
        for n in sizes:
            raw = torch.full((n + 2048,), FILL, dtype=torch.uint8, device="cuda")
            skew = (-raw.data_ptr()) % 1024 + 16
            v = raw[skew: skew + n]
            assert v.data_ptr() % 32 == 16
            bufs.append((raw, v))
        xb, wb, ub, wsb, yb, bb = [v for _, v in bufs]
        xb.copy_(torch.from_numpy(x_q.reshape(-1).view(np.uint8)))
        wb.copy_(torch.from_numpy(w_q.reshape(-1).view(np.uint8)))
        bb.copy_(torch.from_numpy(bias.view(np.uint8)))
        plan.transform_weights(wb, ub)
        plan.conv_forward(xb, ub, bb, yb, wsb)
        assert plan.last_status() == 0
        got = yb.cpu().numpy().view(np.int8).reshape(y_ref.shape)
        assert (got == y_ref).all(), path
