"""Seeded synthetic inputs for the Winograd-aware quantized convolution layer.

This module only *draws tensors*: activations, weights, biases, the Gaussian
perturbation used for "flex" transform matrices, and the table of workload
shapes.  It contains none of the layer's arithmetic (no transform, no
quantizer of a stage, no convolution), so both the CPU oracle's tests and the
CUDA library's tests can feed from it without sharing method code.

The generator is counter based: value i of stream s under seed k is
``splitmix64(k, s, i)`` (Steele, Lea & Flood's SplitMix64 finalizer applied to a
counter), so any element can be produced independently and the bits do not
depend on the host, the thread count or a library's sampler.  Normal deviates
come from Box-Muller in double precision on that uniform stream.

The shapes stand in for the paper's CIFAR-10 ResNet-18 layers (Section 5.1):
the dataset and trained weights are not used; activations are post-ReLU-like
half-normal integer codes and weights are Gaussian, quantized per tensor.
"""
from __future__ import annotations

from dataclasses import dataclass
from fractions import Fraction

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def bits64(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """n 64-bit words: word i = mix(mix(seed, stream) + (offset+i+1)*golden)."""
    with np.errstate(over="ignore"):
        key = _splitmix(np.array([np.uint64(seed) * _GOLDEN + np.uint64(stream)], np.uint64))
        key = _splitmix(key + _GOLDEN)[0]
        ctr = (np.arange(offset + 1, offset + n + 1, dtype=np.uint64)) * _GOLDEN + key
    return _splitmix(ctr)


def uniform(seed: int, stream: int, n: int) -> np.ndarray:
    """Doubles in (0, 1): (top 53 bits + 0.5) / 2^53."""
    return ((bits64(seed, stream, n) >> np.uint64(11)).astype(np.float64) + 0.5) / float(1 << 53)


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """Standard normal deviates by Box-Muller (double precision)."""
    h = (n + 1) // 2
    u1 = uniform(seed, 2 * stream, h)
    u2 = uniform(seed, 2 * stream + 1, h)
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * h, np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n]


def uniform_int8(seed: int, stream: int, shape, lo: int = -127, hi: int = 127) -> np.ndarray:
    n = int(np.prod(shape))
    span = np.uint64(hi - lo + 1)
    v = (bits64(seed, stream, n) >> np.uint64(16)) % span
    return (v.astype(np.int64) + lo).astype(np.int8).reshape(shape)


def halfnormal_codes(seed: int, stream: int, shape, sigma: float = 32.0, hi: int = 127) -> np.ndarray:
    """Post-ReLU-like activation codes: min(hi, round(|N(0, sigma^2)|))."""
    n = int(np.prod(shape))
    v = np.rint(np.abs(normal(seed, stream, n)) * sigma)
    return np.minimum(v, hi).astype(np.int8).reshape(shape)


def gaussian_weight_codes(seed: int, stream: int, shape, sigma: float):
    """Weights ~ N(0, sigma^2), per-tensor symmetric int8 codes.
    Returns (codes int8, scale float32) with scale = max|w| / 127."""
    n = int(np.prod(shape))
    w = normal(seed, stream, n) * sigma
    s = np.float32(np.max(np.abs(w)) / 127.0)
    q = np.clip(np.rint(w / np.float64(s)), -127, 127).astype(np.int8).reshape(shape)
    return q, s


def bias_values(seed: int, stream: int, K: int, sigma: float) -> np.ndarray:
    return (normal(seed, stream, K) * sigma).astype(np.float32)


def flex_perturb(mat32: np.ndarray, seed: int, stream: int, sigma: float = 0.01) -> np.ndarray:
    """'flex' stand-in for learnt transforms: every entry (zeros too) of the
    fp32 Cook-Toom matrix plus sigma*N(0,1), result in fp32."""
    z = normal(seed, stream, mat32.size).reshape(mat32.shape)
    return (mat32.astype(np.float64) + sigma * z).astype(np.float32)


def channel_factors(seed: int, K: int, spread: float = 2.0):
    """Four arrays of K factors, log-uniform in [1/spread, spread]: what per-output-channel
    scales for the weights, the transformed weights, the Hadamard sums and the output are
    multiplied by."""
    out = []
    for j in range(4):
        u = uniform(seed, S_CH + j, K)
        out.append(np.exp((2.0 * u - 1.0) * np.log(spread)).astype(np.float32))
    return out


POINTS = {
    2: [0, 1, -1],
    4: [0, 1, -1, 2, -2],
    6: [0, 1, -1, 2, -2, Fraction(1, 2), Fraction(-1, 2)],
}

# stream ids
S_X, S_W, S_BIAS, S_BT, S_G, S_AT, S_M = 1, 2, 3, 4, 5, 6, 7
S_CH = 8   # per-output-channel scale factors (four consecutive streams)


@dataclass(frozen=True)
class Workload:
    name: str
    seed: int
    N: int
    C: int
    H: int
    W: int
    K: int
    m: int
    flex: bool = False
    fixed_scales: float | None = None   # all six stage scales fixed at this value
    act: str = "halfnormal"             # or "uniform"
    w_sigma: float | None = 0.05        # None: uniform int8 codes


CONFIGS = {
    "cfg1": Workload("cfg1", 1001, 1, 16, 8, 8, 16, 2, fixed_scales=1.0 / 64, act="uniform",
                     w_sigma=None),
    "cfg2": Workload("cfg2", 1002, 64, 64, 32, 32, 64, 2),
    "cfg3": Workload("cfg3", 1003, 256, 256, 8, 8, 256, 4),
    "cfg4": Workload("cfg4", 1004, 128, 128, 16, 16, 128, 6, flex=True),
}


def make_tensors(wl: Workload, N: int | None = None, with_bias: bool = True):
    """x_q, s_x, w_q, s_w, bias for a workload (optionally with a smaller batch)."""
    N = wl.N if N is None else N
    xs = (N, wl.H, wl.W, wl.C)
    ws = (wl.K, 3, 3, wl.C)
    if wl.act == "uniform":
        x_q = uniform_int8(wl.seed, S_X, xs)
    else:
        x_q = halfnormal_codes(wl.seed, S_X, xs)
    if wl.fixed_scales is not None:
        s_x = np.float32(wl.fixed_scales)
    else:
        s_x = np.float32(1.0 / 32.0)
    if wl.w_sigma is None:
        w_q = uniform_int8(wl.seed, S_W, ws)
        s_w = np.float32(wl.fixed_scales if wl.fixed_scales is not None else 1.0 / 64)
    else:
        w_q, s_w = gaussian_weight_codes(wl.seed, S_W, ws, wl.w_sigma)
    bias = None
    if with_bias:
        # a bias of the order of one output standard deviation
        sig = float(s_x) * 32.0 * float(s_w) * 40.0 * np.sqrt(9.0 * wl.C) * 0.25
        bias = bias_values(wl.seed, S_BIAS, wl.K, sig)
    return x_q, s_x, w_q, s_w, bias


def resnet18_layers(seed: int = 1005, batch: int = 256):
    """The sixteen 3x3 convolutions of a CIFAR-shaped ResNet-18 body (widths
    64/128/256/512 at 32/16/8/4 pixels).  Stride-2 layers carry m = 0 (they are
    not Winograd layers); every stride-1 layer draws its tile size m from
    {2, 4, 6} with the seed, mimicking a searched per-layer assignment
    (Section 4).  Returns a list of dicts."""
    plan = []
    widths = [64, 128, 256, 512]
    size = 32
    cin = 64
    for si, wdt in enumerate(widths):
        for li in range(4):
            stride = 2 if (si > 0 and li == 0) else 1
            plan.append(dict(C=cin, K=wdt, H=size, W=size, stride=stride))
            if stride == 2:
                size //= 2
            cin = wdt
    draws = bits64(seed, S_M, len(plan))
    out = []
    for i, p in enumerate(plan):
        m = 0 if p["stride"] == 2 else [2, 4, 6][int(draws[i] % np.uint64(3))]
        out.append(dict(index=i, N=batch, m=m, **p))
    return out
