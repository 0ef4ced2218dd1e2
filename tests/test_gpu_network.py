"""cfg5: the sixteen 3x3 convolutions of a CIFAR-shaped ResNet-18 body chained
conv -> ReLU -> conv in int8, tile size per stride-1 layer drawn from a seed
(mimicking a searched per-layer assignment, paper Section 4).  Stride-2 layers
are direct convolutions (oracle: integer definition; GPU: the library's direct kernel).  Every Winograd layer's GPU output must
equal the oracle's byte for byte, both when fed the oracle's activations and
when fed the GPU chain's own."""
import numpy as np
import pytest

import oracle
import wino_inputs as wi
from helpers import matrices
from oracle import Layer, Quant
from oracle.calibrate import calibrate

pytestmark = pytest.mark.gpu


def _weights(seed, idx, K, C):
    return wi.gaussian_weight_codes(seed, 100 + idx, (K, 3, 3, C), float(np.sqrt(2.0 / (9 * C))))


def _run_chain(batch, per_channel_weights=False):
    from gpu_helpers import gpu_run
    seed = 1005
    layers = wi.resnet18_layers(seed, batch)
    x_ref = wi.halfnormal_codes(seed, wi.S_X, (batch, 32, 32, 64))
    x_gpu = x_ref.copy()
    s_x = float(np.float32(1.0 / 32.0))
    seen_m = set()
    for spec in layers:
        w_q, s_w = _weights(seed, spec["index"], spec["K"], spec["C"])
        if spec["stride"] == 2:
            acc = oracle.direct_conv_i32(x_ref, w_q, stride=2)
            real_max = float(np.abs(acc).max()) * s_x * float(s_w)
            q_Y = Quant(scale=float(np.float32(real_max / 127.0)), qmin=0)
            s_w_K = s_in_K = None
            if per_channel_weights:
                s_w_K = (np.float32(s_w) * wi.channel_factors(seed + spec["index"], spec["K"], 1.5)[0]).astype(np.float32)
                s_in_K = s_w_K.astype(np.float64) * np.float64(np.float32(s_x))
            x_ref = oracle.requantize_acc(acc, s_x * float(s_w), q_Y, s_in_K=s_in_K)
            # the GPU chain runs its strided layers with the library's direct convolution
            import torch
            from paper_2002_10711_b200 import binding
            xd = torch.from_numpy(x_gpu).cuda()
            wd = torch.from_numpy(w_q).cuda()
            yd = torch.empty(x_ref.shape, dtype=torch.int8, device="cuda")
            binding.direct_conv_forward(batch, spec["C"], spec["H"], spec["W"], spec["K"], 2,
                                        Quant(scale=s_x), Quant(scale=float(s_w)), q_Y, xd, wd, None, yd,
                                        s_w_K_dev=None if s_w_K is None else torch.from_numpy(s_w_K).cuda())
            torch.cuda.synchronize()
            x_gpu = yd.cpu().numpy()
            assert (x_gpu == x_ref).all(), f"layer {spec['index']} (direct, stride 2) differs"
            s_x = q_Y.scale
            continue
        m = spec["m"]
        seen_m.add(m)
        BT, G, AT = matrices(m)
        L = Layer(batch, spec["C"], spec["H"], spec["W"], spec["K"], m, BT, G, AT)
        L.q_x = Quant(scale=s_x)
        L.q_w = Quant(scale=float(s_w))
        L.q_Y = Quant(qmin=0)
        L = calibrate(L, x_ref, w_q, None)
        if per_channel_weights:
            # weights, transformed weights and Hadamard sums scaled per output channel, activations per
            # layer (the next layer sums over these channels, so its input has one scale)
            f_w, f_U, f_M, _ = wi.channel_factors(seed + spec["index"], spec["K"], 1.5)
            L.s_w_K = (np.float32(L.q_w.scale) * f_w).astype(np.float32)
            L.s_U_K = (np.float32(L.q_U.scale) * f_U).astype(np.float32)
            L.s_M_K = (np.float32(L.q_M.scale) * f_M).astype(np.float32)
        y_ref = oracle.forward(L, x_ref, w_q)
        g1 = gpu_run(L, x_ref, w_q, None)
        assert (g1["y"] == y_ref).all(), f"layer {spec['index']} (oracle-fed) differs"
        g2 = gpu_run(L, x_gpu, w_q, None)
        assert (g2["y"] == y_ref).all(), f"layer {spec['index']} (GPU-fed) differs"
        assert y_ref.min() >= 0 and y_ref.max() > 0
        x_ref, x_gpu, s_x = y_ref, g2["y"], L.q_Y.scale
    return seen_m


def test_resnet18_chain_small_batch():
    seen = _run_chain(4)
    assert seen == {2, 4, 6}


def test_resnet18_chain_with_per_channel_weight_scales():
    seen = _run_chain(4, per_channel_weights=True)
    assert seen == {2, 4, 6}


def test_resnet18_chain_full_batch():
    # the configuration as stated: batch 256, all sixteen layers
    seen = _run_chain(256)
    assert seen == {2, 4, 6}


@pytest.mark.parametrize("index", [0, 13])
def test_resnet18_layer_full_batch(index):
    from gpu_helpers import gpu_run
    spec = wi.resnet18_layers(1005, 256)[index]
    assert spec["stride"] == 1
    x_q = wi.halfnormal_codes(1005 + index, wi.S_X, (256, spec["H"], spec["W"], spec["C"]))
    w_q, s_w = _weights(1005, index, spec["K"], spec["C"])
    BT, G, AT = matrices(spec["m"])
    L = Layer(256, spec["C"], spec["H"], spec["W"], spec["K"], spec["m"], BT, G, AT)
    L.q_x = Quant(scale=1.0 / 32)
    L.q_w = Quant(scale=float(s_w))
    L.q_Y = Quant(qmin=0)
    L = calibrate(L, x_q, w_q, None)
    y_ref = oracle.forward(L, x_q, w_q)
    g = gpu_run(L, x_q, w_q, None)
    assert (g["y"] == y_ref).all()
