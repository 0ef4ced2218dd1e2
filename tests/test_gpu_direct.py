"""Direct int8 3x3 convolution on the GPU (stride 1 and 2) against the oracle's
integer direct convolution and output quantizer: bit-exact int8 codes."""
import numpy as np
import pytest

import oracle
import wino_inputs as wi
from oracle import Quant

pytestmark = pytest.mark.gpu


def _run(N, C, H, W, K, stride, q_x, q_w, q_Y, x_q, w_q, bias, out_dtype=0):
    import torch
    from paper_2002_10711_b200 import binding
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    x = torch.from_numpy(x_q).cuda()
    w = torch.from_numpy(w_q).cuda()
    b = None if bias is None else torch.from_numpy(bias).cuda()
    y = torch.empty((N, Ho, Wo, K), dtype=torch.float32 if out_dtype else torch.int8, device="cuda")
    binding.direct_conv_forward(N, C, H, W, K, stride, q_x, q_w, q_Y, x, w, b, y, out_dtype=out_dtype)
    torch.cuda.synchronize()
    return y.cpu().numpy()


# the second row of shapes runs on the tensor cores at stride 1 without zero points (C % 64 == 0,
# K % 32 == 0): ragged tiles, tiles spanning several images, 64- and 128-byte channel blocks
@pytest.mark.parametrize("shape", [(2, 16, 9, 7, 8), (1, 64, 32, 32, 128), (3, 4, 1, 1, 4), (2, 128, 16, 16, 256),
                                   (1, 20, 6, 11, 12),
                                   (3, 128, 8, 8, 64), (5, 64, 4, 4, 96), (1, 256, 5, 19, 32), (2, 192, 1, 1, 64),
                                   (1, 512, 4, 4, 512), (2, 64, 9, 7, 32),
                                   (2, 128, 7, 9, 32), (20, 64, 16, 16, 64),   # weights resident in shared memory, several items per block
                                   (2, 3, 32, 32, 64), (2, 5, 7, 9, 6)])   # any channel count: byte-wise kernel
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("variant", ["plain", "relu_bias", "zero_points"])
def test_direct_conv_matches_oracle(shape, stride, variant):
    N, C, H, W, K = shape
    x_q = wi.halfnormal_codes(5000 + C, 1, (N, H, W, C))
    w_q, s_w = wi.gaussian_weight_codes(5000 + K, 2, (K, 3, 3, C), 0.05)
    s_x = float(np.float32(1 / 32))
    z_x = z_w = 0
    bias = None
    q_Y = Quant()
    if variant == "relu_bias":
        bias = wi.bias_values(5000, 3, K, 0.5)
        q_Y = Quant(qmin=0)
    if variant == "zero_points":
        z_x, z_w = 4, -3
        q_Y = Quant(zero_point=6)
    acc = oracle.direct_conv_i32(x_q, w_q, z_x=z_x, z_w=z_w, stride=stride)
    s_in = s_x * float(s_w)
    q_Y.scale = float(np.float32(max(float(np.abs(acc).max()) * s_in, 1e-6) / 127.0))
    want = oracle.requantize_acc(acc, s_in, q_Y, bias)
    got = _run(N, C, H, W, K, stride, Quant(scale=s_x, zero_point=z_x), Quant(scale=float(s_w), zero_point=z_w),
               q_Y, x_q, w_q, bias)
    assert got.shape == want.shape and (got == want).all()
    assert want.size < 100 or len(np.unique(want)) > 3
    from paper_2002_10711_b200 import binding
    assert binding.direct_last_status() == 0


def test_direct_conv_float_output():
    N, C, H, W, K = 2, 32, 10, 9, 16
    x_q = wi.halfnormal_codes(5100, 1, (N, H, W, C))
    w_q, s_w = wi.gaussian_weight_codes(5100, 2, (K, 3, 3, C), 0.05)
    bias = wi.bias_values(5100, 3, K, 0.5)
    s_x = float(np.float32(1 / 32))
    acc = oracle.direct_conv_i32(x_q, w_q, stride=2)
    s_in = np.float32(s_x * float(s_w))
    want = acc.astype(np.float32).astype(np.float64) * np.float64(s_in) + bias.astype(np.float64)
    got = _run(N, C, H, W, K, 2, Quant(scale=s_x), Quant(scale=float(s_w)), Quant(), x_q, w_q, bias, out_dtype=1)
    assert float(np.abs(got - want).max()) <= 1e-4 * float(np.abs(want).max())


def test_direct_conv_float_output_tensor_core_path():
    N, C, H, W, K = 2, 64, 10, 9, 32
    x_q = wi.halfnormal_codes(5200, 1, (N, H, W, C))
    w_q, s_w = wi.gaussian_weight_codes(5200, 2, (K, 3, 3, C), 0.05)
    bias = wi.bias_values(5200, 3, K, 0.5)
    s_x = float(np.float32(1 / 32))
    acc = oracle.direct_conv_i32(x_q, w_q, stride=1)
    s_in = np.float32(s_x * float(s_w))
    want = acc.astype(np.float32).astype(np.float64) * np.float64(s_in) + bias.astype(np.float64)
    got = _run(N, C, H, W, K, 1, Quant(scale=s_x), Quant(scale=float(s_w)), Quant(), x_q, w_q, bias, out_dtype=1)
    assert float(np.abs(got - want).max()) <= 1e-4 * float(np.abs(want).max())


def test_direct_conv_resnet_layer_shapes_at_batch():
    # the layer shapes of the ResNet-18 body at a batch that fills the GPU several times over
    for (N, C, H, W, K) in [(32, 64, 32, 32, 64), (32, 256, 8, 8, 256)]:
        x_q = wi.halfnormal_codes(5300 + C, 1, (N, H, W, C))
        w_q, s_w = wi.gaussian_weight_codes(5300 + K, 2, (K, 3, 3, C), 0.05)
        s_x = float(np.float32(1 / 32))
        acc = oracle.direct_conv_i32(x_q, w_q, stride=1)
        s_in = s_x * float(s_w)
        q_Y = Quant(qmin=0)
        q_Y.scale = float(np.float32(float(np.abs(acc).max()) * s_in / 127.0))
        bias = wi.bias_values(5300, 3, K, 0.5)
        want = oracle.requantize_acc(acc, s_in, q_Y, bias)
        got = _run(N, C, H, W, K, 1, Quant(scale=s_x), Quant(scale=float(s_w)), q_Y, x_q, w_q, bias)
        assert (got == want).all()


def test_direct_conv_tensor_core_path_writes_nothing_outside_y():
    # ragged tiles (W = 19 > 16, H = 5 < 8) and a tile that spans images past N: the output sits
    # between guard bands that must keep their pattern
    import torch
    from paper_2002_10711_b200 import binding
    for (N, C, H, W, K) in [(1, 64, 5, 19, 32), (3, 128, 8, 8, 64), (5, 64, 4, 4, 96)]:
        x_q = wi.halfnormal_codes(5400 + C, 1, (N, H, W, C))
        w_q, s_w = wi.gaussian_weight_codes(5400 + K, 2, (K, 3, 3, C), 0.05)
        s_x = float(np.float32(1 / 32))
        acc = oracle.direct_conv_i32(x_q, w_q, stride=1)
        s_in = s_x * float(s_w)
        q_Y = Quant(scale=float(np.float32(float(np.abs(acc).max()) * s_in / 127.0)))
        want = oracle.requantize_acc(acc, s_in, q_Y, None)
        guard = 4096
        nbytes = N * H * W * K
        arena = torch.full((guard + nbytes + guard,), 0x5A, dtype=torch.uint8, device="cuda")
        y = arena[guard:guard + nbytes].view(torch.int8).view(N, H, W, K)
        assert y.data_ptr() % 32 == 0
        x = torch.from_numpy(x_q).cuda()
        w = torch.from_numpy(w_q).cuda()
        binding.direct_conv_forward(N, C, H, W, K, 1, Quant(scale=s_x), Quant(scale=float(s_w)), q_Y, x, w, None, y)
        torch.cuda.synchronize()
        assert binding.direct_last_status() == 0
        a = arena.cpu().numpy()
        assert (a[:guard] == 0x5A).all() and (a[guard + nbytes:] == 0x5A).all()
        assert (a[guard:guard + nbytes].view(np.int8).reshape(N, H, W, K) == want).all()


def test_direct_conv_argument_checks():
    from paper_2002_10711_b200 import binding
    q = Quant()
    with pytest.raises(binding.WinoError) as e:
        binding.direct_conv_forward(1, 16, 8, 8, 16, 3, q, q, q, 16, 16, None, 16, stream=0)
    assert e.value.code == binding.ERR_INVALID
    with pytest.raises(binding.WinoError) as e:
        binding.direct_conv_forward(1, 8, 8, 8, 16, 1, q, q, q, 16, 24, None, 16, stream=0)   # w not 16-byte aligned
    assert e.value.code == binding.ERR_ALIGNMENT


# per-output-channel scales (Section 7) on every direct-convolution kernel: tensor cores
# (stride 1 and 2), integer dot products, byte-wise
@pytest.mark.parametrize("shape,stride", [((2, 64, 9, 7, 32), 1), ((3, 128, 8, 8, 64), 2), ((1, 256, 5, 19, 288), 1),
                                          ((20, 64, 16, 16, 64), 2), ((2, 128, 7, 9, 32), 1),
                                          ((2, 16, 9, 7, 8), 1), ((1, 20, 6, 11, 12), 2), ((2, 3, 16, 16, 6), 1)])
@pytest.mark.parametrize("which", ["both", "weights_only", "output_only"])
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_direct_conv_per_channel_scales(shape, stride, which, out_dtype):
    import torch
    from paper_2002_10711_b200 import binding
    N, C, H, W, K = shape
    x_q = wi.halfnormal_codes(5600 + C, 1, (N, H, W, C))
    w_q, s_w = wi.gaussian_weight_codes(5600 + K, 2, (K, 3, 3, C), 0.05)
    bias = wi.bias_values(5600, 3, K, 0.5)
    s_x = np.float32(1 / 32)
    f_w, _, _, f_Y = wi.channel_factors(5600 + K, K, 3.0)
    acc = oracle.direct_conv_i32(x_q, w_q, stride=stride)
    s_in = float(np.float64(s_x) * np.float64(s_w))
    q_Y = Quant(qmin=-120, zero_point=2)
    q_Y.scale = float(np.float32(max(float(np.abs(acc).max()) * s_in, 1e-6) / 127.0))
    s_w_K = (np.float32(s_w) * f_w).astype(np.float32) if which != "output_only" else None
    s_Y_K = (np.float32(q_Y.scale) * f_Y).astype(np.float32) if which != "weights_only" else None
    s_in_K = None if s_w_K is None else s_w_K.astype(np.float64) * np.float64(s_x)
    dev = lambda a: None if a is None else torch.from_numpy(a).cuda()
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    y = torch.empty((N, Ho, Wo, K), dtype=torch.float32 if out_dtype else torch.int8, device="cuda")
    binding.direct_conv_forward(N, C, H, W, K, stride, Quant(scale=float(s_x)), Quant(scale=float(s_w)), q_Y,
                                dev(x_q), dev(w_q), dev(bias), y, out_dtype=out_dtype,
                                s_w_K_dev=dev(s_w_K), s_Y_K_dev=dev(s_Y_K))
    torch.cuda.synchronize()
    assert binding.direct_last_status() == 0
    got = y.cpu().numpy()
    if out_dtype == 0:
        want = oracle.requantize_acc(acc, s_in, q_Y, bias, s_in_K=s_in_K, s_Y_K=s_Y_K)
        assert (got == want).all()
        assert len(np.unique(want)) > 10
    else:
        # float output: fmaf(acc, (float)(s_x * s_w[k]), bias[k]), exactly rounded once
        s_k = (s_in_K if s_in_K is not None else np.full(K, s_in)).astype(np.float32).astype(np.float64)
        exact = acc.astype(np.float64) * s_k + bias.astype(np.float64)
        assert (got == exact.astype(np.float32)).all()
