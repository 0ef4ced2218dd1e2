"""Per-layer latency table on the current GPU: for each 3x3 layer shape, the time
of the direct int8 convolution and of the Winograd-aware layer with m = 2, 4, 6.
This is the lookup table a latency-aware search over convolution algorithms
needs (paper: Section 4, "each candidate operation comes with its respective
latency"); the paper filled it on Arm cores.

    python -m paper_2002_10711_b200.latency_table [--batch 256] [--channels 256] [--strided]

The direct convolution is the library's implicit GEMM on the tensor cores (stride 1,
channel counts that are multiples of 64 / 32; other layers run on the integer ALUs).

Prints one JSON object per shape.  Steady-state time per call: the call is
captured in a CUDA graph on rotating buffers and timed with CUDA events.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding, cook_toom

RESNET18_CIFAR = [(64, 32), (128, 16), (256, 8), (512, 4)]   # (channels, spatial size)


def _time_graph(fn, reps=10, inner=8):
    for i in range(3):
        fn(i)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(inner):
                fn(i)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * inner)


def layer_latencies(N, C, H, W, K, device="cuda:0", sets=8):
    """Microseconds per call for {"direct", "F2", "F4", "F6"} on random int8 data (the
    kernels have no data-dependent control flow, so the values do not matter)."""
    dev = torch.device(device)
    gen = torch.Generator(device="cpu").manual_seed(1)
    xs = [torch.randint(0, 127, (N, H, W, C), dtype=torch.int8, generator=gen).to(dev) for _ in range(sets)]
    w = torch.randint(-127, 127, (K, 3, 3, C), dtype=torch.int8, generator=gen).to(dev)
    ys = [torch.empty((N, H, W, K), dtype=torch.int8, device=dev) for _ in range(sets)]
    q = dict(scale=0.05)
    out = {}
    out["direct"] = _time_graph(lambda i: binding.direct_conv_forward(
        N, C, H, W, K, 1, q, q, dict(scale=4.0), xs[i % sets], w, None, ys[i % sets]))
    for m in (2, 4, 6):
        BT, G, AT = cook_toom(m)
        try:
            plan = binding.Plan(N, C, H, W, K, m, BT, G, AT, q, q, dict(scale=0.5), dict(scale=0.02),
                                dict(scale=1.0), dict(scale=4.0))
        except binding.WinoError:
            out[f"F{m}"] = None
            continue
        Uq = torch.empty(plan.weight_bytes, dtype=torch.int8, device=dev)
        ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device=dev)
        plan.transform_weights(w, Uq)
        out[f"F{m}"] = _time_graph(lambda i: plan.conv_forward(xs[i % sets], Uq, None, ys[i % sets], ws))
        assert plan.last_status() == 0
    return out


def strided_latency(N, C, H, W, K, device="cuda:0", sets=8):
    """Microseconds per call of the stride-2 direct convolution C -> K on an H x W input."""
    dev = torch.device(device)
    gen = torch.Generator(device="cpu").manual_seed(2)
    xs = [torch.randint(0, 127, (N, H, W, C), dtype=torch.int8, generator=gen).to(dev) for _ in range(sets)]
    w = torch.randint(-127, 127, (K, 3, 3, C), dtype=torch.int8, generator=gen).to(dev)
    ys = [torch.empty((N, (H - 1) // 2 + 1, (W - 1) // 2 + 1, K), dtype=torch.int8, device=dev)
          for _ in range(sets)]
    q = dict(scale=0.05)
    t = _time_graph(lambda i: binding.direct_conv_forward(
        N, C, H, W, K, 2, q, q, dict(scale=4.0), xs[i % sets], w, None, ys[i % sets]))
    assert binding.direct_last_status() == 0
    return t


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--channels", type=int, default=0, help="only the layer shape of this width")
    ap.add_argument("--strided", action="store_true",
                    help="also the network's three stride-2 layers (direct convolution only)")
    args = ap.parse_args()
    if args.strided:
        for (C, S), (K, _) in zip(RESNET18_CIFAR[:-1], RESNET18_CIFAR[1:]):
            print(json.dumps({"N": args.batch, "C": C, "K": K, "H": S, "W": S, "stride": 2,
                              "us": {"direct": round(strided_latency(args.batch, C, S, S, K), 1)}}), flush=True)
    for C, S in RESNET18_CIFAR:
        if args.channels and C != args.channels:
            continue
        lat = layer_latencies(args.batch, C, S, S, C)
        best = min((v, k) for k, v in lat.items() if v is not None)[1]
        print(json.dumps({"N": args.batch, "C": C, "K": C, "H": S, "W": S,
                          "us": {k: (None if v is None else round(v, 1)) for k, v in lat.items()},
                          "fastest": best}), flush=True)


if __name__ == "__main__":
    main()
