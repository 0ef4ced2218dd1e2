"""wino_conv_forward_static: the forward pass for callers that cannot allocate
a workspace (a plug-in whose host framework owns all device memory, a serving
loop that must not touch the CUDA allocator).  It has to give exactly the bytes
of wino_conv_forward, call after call, while sharing one static scratch array
between plans; and it has to refuse a layer whose scratch does not fit.

Collected last on purpose: a failure here must not hide any other test."""
import numpy as np
import pytest

import wino_inputs as wi
from helpers import build_layer, small

pytestmark = pytest.mark.gpu


def _run_both(L, x_q, w_q, bias, path=0):
    import torch
    from paper_2002_10711_b200 import binding
    from paper_2002_10711_b200.layer import WinogradConv
    plan = binding.Plan.from_layer(L, path=path)
    assert plan.workspace_bytes <= binding.STATIC_SCRATCH_BYTES
    conv = WinogradConv(plan)
    conv.load_weights(w_q, bias)
    x = torch.from_numpy(np.ascontiguousarray(x_q)).cuda()
    y_ws = conv.forward(x)                       # existing entry point, caller's workspace
    assert plan.last_status() == 0
    outs = []
    for _ in range(2):                           # two calls in a row on the shared array
        y = conv.empty_output()
        y.fill_(0)
        plan.conv_forward_static(x, conv.Uq, conv.bias, y)
        assert plan.last_status() == 0
        outs.append(y.cpu().numpy())
    return y_ws.cpu().numpy(), outs


@pytest.mark.parametrize("name,N", [("cfg3", 64), ("cfg4", 16), ("cfg2", 4)])
def test_static_scratch_matches_workspace_entry_point(name, N):
    wl = small(wi.CONFIGS[name], N=N)
    L, x_q, w_q, bias = build_layer(wl)
    want, outs = _run_both(L, x_q, w_q, bias)
    assert np.abs(want).max() > 0
    for got in outs:
        assert (got == want).all()               # int8 output: bit-exact, as in the parity tests


def test_two_plans_share_the_array_back_to_back():
    a = build_layer(small(wi.CONFIGS["cfg3"], N=32))
    b = build_layer(small(wi.CONFIGS["cfg4"], N=8))
    for _ in range(2):
        for L, x_q, w_q, bias in (a, b):
            want, outs = _run_both(L, x_q, w_q, bias)
            assert all((g == want).all() for g in outs)


def test_pointer_based_path_and_float_output():
    wl = small(wi.CONFIGS["cfg3"], N=8, C=48, K=80)
    L, x_q, w_q, bias = build_layer(wl, out_dtype=1)
    want, outs = _run_both(L, x_q, w_q, bias)
    tol = 1e-4 * float(np.abs(want).max())      # float output: the parity tests' tolerance
    for got in outs:
        assert float(np.abs(got - want).max()) <= tol


def test_oversized_layer_is_refused():
    import torch
    from paper_2002_10711_b200 import binding
    L, x_q, w_q, bias = build_layer(wi.CONFIGS["cfg2"])      # 33.6 MB of scratch
    plan = binding.Plan.from_layer(L)
    assert plan.workspace_bytes > binding.STATIC_SCRATCH_BYTES
    x = torch.from_numpy(x_q).cuda()
    Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device="cuda")
    y = torch.empty((L.N, L.H, L.W, L.K), dtype=torch.int8, device="cuda")
    before = plan.launch_count
    with pytest.raises(binding.WinoError) as e:
        plan.conv_forward_static(x, Uq, None, y)
    assert e.value.code == binding.ERR_WORKSPACE
    assert plan.launch_count == before
