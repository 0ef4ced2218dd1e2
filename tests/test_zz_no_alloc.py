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


def _run_both(L, x_q, w_q, bias, path=0, side_stream=False):
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
    ys = [conv.empty_output().fill_(0) for _ in range(2)]
    stream = torch.cuda.Stream() if side_stream else torch.cuda.current_stream()
    # first use on this device (address look-up, code loading) happens here, untimed and unmeasured
    plan.conv_forward_static(x, conv.Uq, conv.bias, conv.empty_output(), stream=stream)
    assert plan.last_status(stream) == 0
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    launches_before = plan.launch_count
    outs = []
    for y in ys:                                 # two calls in a row on the shared array
        plan.conv_forward_static(x, conv.Uq, conv.bias, y, stream=stream)
        assert plan.last_status(stream) == 0
    # the promise "allocates nothing": free device memory is what it was
    assert torch.cuda.mem_get_info()[0] == free_before
    per_call = 1 if plan.path in (binding.PATH_SMALLC, binding.PATH_FUSED_F2) else 3
    assert plan.launch_count - launches_before == 2 * per_call
    outs = [y.cpu().numpy() for y in ys]
    return y_ws.cpu().numpy(), outs


# cfg2 at a small batch: once on the path the plan picks (single-kernel F2, no scratch at
# all) and once pinned to the staged path so that the static array is what carries V_q / m_q
@pytest.mark.parametrize("name,N,path", [("cfg3", 64, 0), ("cfg4", 16, 0), ("cfg2", 4, 0), ("cfg2", 4, 1)])
def test_static_scratch_matches_workspace_entry_point(name, N, path):
    wl = small(wi.CONFIGS[name], N=N)
    L, x_q, w_q, bias = build_layer(wl)
    want, outs = _run_both(L, x_q, w_q, bias, path=path)
    assert np.abs(want).max() > 0
    for got in outs:
        assert (got == want).all()               # int8 output: bit-exact, as in the parity tests


def test_static_scratch_on_a_side_stream():
    wl = small(wi.CONFIGS["cfg3"], N=16)
    L, x_q, w_q, bias = build_layer(wl)
    want, outs = _run_both(L, x_q, w_q, bias, side_stream=True)
    for got in outs:
        assert (got == want).all()


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


def _run_both_big(L, x_q, w_q, bias, plan):
    import torch
    from paper_2002_10711_b200.layer import WinogradConv
    conv = WinogradConv(plan)
    conv.load_weights(w_q, bias)
    x = torch.from_numpy(np.ascontiguousarray(x_q)).cuda()
    want = conv.forward(x).cpu().numpy()
    y = conv.empty_output().fill_(0)
    plan.conv_forward_static(x, conv.Uq, conv.bias, y)
    assert plan.last_status() == 0
    return want, y.cpu().numpy()


def test_oversized_layer_is_refused_on_a_staged_path_only():
    import torch
    from paper_2002_10711_b200 import binding
    L, x_q, w_q, bias = build_layer(wi.CONFIGS["cfg2"])      # 33.6 MB of scratch when staged
    plan = binding.Plan.from_layer(L)
    assert plan.workspace_bytes > binding.STATIC_SCRATCH_BYTES
    # the plan's own choice for this layer is the single-kernel F2 path: no scratch, accepted
    assert plan.path == binding.PATH_FUSED_F2
    want, outs = _run_both_big(L, x_q, w_q, bias, plan)
    assert (outs == want).all()
    plan.force_path(binding.PATH_STAGED_TC)
    x = torch.from_numpy(x_q).cuda()
    Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device="cuda")
    y = torch.empty((L.N, L.H, L.W, L.K), dtype=torch.int8, device="cuda")
    before = plan.launch_count
    with pytest.raises(binding.WinoError) as e:
        plan.conv_forward_static(x, Uq, None, y)
    assert e.value.code == binding.ERR_WORKSPACE
    assert plan.launch_count == before
