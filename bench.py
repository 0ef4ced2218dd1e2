#!/usr/bin/env python
"""Benchmark of the Winograd-aware quantized conv forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one forward pass of the layer (input transform, Hadamard-stage
GEMMs, output transform, all quantizers) over one batch of the workload, with
the transformed weights resident, as the paper treats them (Section 3.1: the
weight transform is done once and reused by every inference); it is timed
separately and reported beside it.  The metric is effective direct-convolution-
equivalent int8 TOPS: 2*N*H*W*K*C*9 operations per step over the measured time.

Prints ONE JSON line (rank 0).  With torchrun (N > 1) every rank processes its
own batch (weak scaling, no collective on the data path); time is the max over
ranks, value the sum of work over that time.

Beside the contract's keys the line carries: `stages` (each kernel of a step
timed alone), `roofline` (the dominant kernel; `traffic` = its DRAM bytes per
launch from profiles/traffic.json while the digest stored there matches the CUDA
sources, else null), `layer_roofline` (whole step against max(t_MMA, t_HBM), and
`three_term` with the ALU issue bound from the same counters), `warm_l2` (every
step on one buffer set), `single_launch` (the one-kernel layer path on the same
workload), `other_configs` (cfg2, cfg4 and the Winograd layers of the ResNet-18
body, one row each), `overlapped_steps`, `int8_mma_probe_TOPS`,
`weight_transform`, `e2e`, `cpu_baseline`, `clocks`.  `--path P` forces a path of
the library, `--no-other-configs` and `--no-cpu-baseline` shorten the run (used
for profiler captures).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import wino_inputs as wi  # noqa: E402

PATH_NAMES = {1: "staged_tc", 2: "staged_dp4a", 3: "smallc", 4: "staged_tc_ptr", 5: "fused_f2",
              6: "staged_tc_mma", 7: "fused_layer"}


def csrc_digest():
    """SHA-256 over the CUDA sources: identifies the kernels a profiler capture belongs to."""
    import hashlib
    root = os.path.join(ROOT, "paper_2002_10711_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(root)):
        if name.endswith((".cu", ".cuh", ".h")):
            h.update(name.encode())
            h.update(open(os.path.join(root, name), "rb").read())
    return h.hexdigest()


def load_counters():
    """profiles/traffic.json: per-kernel ncu counters of the cfg3 workload (DRAM bytes and
    warp instructions per launch) with the digest of the sources they were taken from.
    Returns {} when the sources have changed since (stale counters are not reported)."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return {}
    d = json.load(open(path))
    return d.get("kernels", {}) if d.get("csrc_sha256") == csrc_digest() else {}

METRIC = "effective direct-conv-equivalent int8 TOPS (Winograd-aware quantized 3x3 conv forward)"
UNIT = "TOPS"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


def direct_ops(wl, N):
    return 2.0 * N * wl.H * wl.W * wl.K * wl.C * 9


def wino_ops(wl, N):
    t = wl.m + 2
    T = N * (-(-wl.H // wl.m)) * (-(-wl.W // wl.m))
    return 2.0 * T * t * t * wl.C * wl.K


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed
    region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [v.strip() for v in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------
def run_reference(args, wl):
    """The CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    from helpers import build_layer
    L, x_q, w_q, bias = build_layer(wl)
    Uq = oracle.weight_stage(L, w_q)
    for _ in range(min(args.warmup, 2)):
        oracle.forward(L, x_q, U_q=Uq, bias=bias)
    steps = min(args.steps, 20)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.forward(L, x_q, U_q=Uq, bias=bias)
    dt = (time.perf_counter() - t0) / steps
    value = direct_ops(wl, wl.N) / dt / 1e12
    cores = oracle.num_threads()
    sample = f"full batch N={wl.N} per step, {steps} steps"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "config": workload_config(wl, "host memory (CPU oracle)"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(wl, l2_note):
    return {"workload": f"{wl.name}: ResNet-18 CIFAR layer N={wl.N} C=K={wl.C} H=W={wl.H} "
                        f"F({wl.m}x{wl.m},3x3) int8, "
                        + ("all stage scales fixed" if wl.fixed_scales is not None
                           else "per-stage max-abs scales"),
            "N": wl.N, "C": wl.C, "K": wl.K, "H": wl.H, "W": wl.W, "m": wl.m, "l2": l2_note}


def aggregate(ms_local: float, units_local: float, dist=None):
    """Max time over ranks, summed work.  `dist`: torch.distributed or None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_local, units_local
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def time_layer_quick(binding, cook_toom, torch, dev, N, C, H, W, K, m, flex_seed=None, path=0,
                     steps=96, channel_scales=False):
    """Steady-state microseconds per forward call of one layer shape on rotating buffers
    (more bytes than L2), from a CUDA graph, with fixed stage scales: the kernels have no
    data-dependent control flow, so for timing the values and scales do not matter.
    Returns (us, path) or (None, reason)."""
    BT, G, AT = cook_toom(m)
    if flex_seed is not None:
        BT = wi.flex_perturb(BT, flex_seed, wi.S_BT)
        G = wi.flex_perturb(G, flex_seed, wi.S_G)
        AT = wi.flex_perturb(AT, flex_seed, wi.S_AT)
    q = lambda sc: dict(scale=sc)
    try:
        plan = binding.Plan(N, C, H, W, K, m, BT, G, AT, q(1 / 32), q(0.004), q(0.5), q(0.01),
                            q(30.0), q(100.0), path=path)
        if channel_scales:   # per-output-channel scales for w, U, M and y (seeded factors)
            f_w, f_U, f_M, f_Y = wi.channel_factors(7, K)
            plan.set_channel_scales(0.004 * f_w, 0.01 * f_U, 30.0 * f_M, 100.0 * f_Y)
    except binding.WinoError as e:
        return None, str(e)
    xb, yb = N * H * W * C, N * H * W * K
    R = max(2, int(np.ceil(1.5 * 126e6 / (xb + yb + plan.weight_bytes))))
    gen = torch.Generator(device="cpu").manual_seed(7)
    x0 = torch.randint(0, 127, (N, H, W, C), dtype=torch.int8, generator=gen).to(dev)
    w = torch.randint(-127, 127, (K, 3, 3, C), dtype=torch.int8, generator=gen).to(dev)
    xs = [x0.clone() for _ in range(R)]
    ys = [torch.empty((N, H, W, K), dtype=torch.int8, device=dev) for _ in range(R)]
    Us = [torch.empty(plan.weight_bytes, dtype=torch.int8, device=dev) for _ in range(R)]
    ws = torch.empty(max(plan.workspace_bytes, 16), dtype=torch.uint8, device=dev)
    for U in Us:
        plan.transform_weights(w, U)

    def step(i):
        j = i % R
        plan.conv_forward(xs[j], Us[j], None, ys[j], ws)

    for i in range(3):
        step(i)
    torch.cuda.synchronize()
    inner = max(2 * R, 8)
    side = torch.cuda.Stream(device=dev)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for i in range(inner):
                step(i)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    reps = max(1, steps // inner)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    if plan.last_status() != 0:
        return None, "device status"
    return e0.elapsed_time(e1) * 1e3 / (reps * inner), plan.path


def layer_row(peaks, name, N, C, H, W, K, m, us, path):
    t = m + 2
    T = N * (-(-H // m)) * (-(-W // m))
    d_ops = 2.0 * N * H * W * K * C * 9
    w_ops = 2.0 * T * t * t * C * K
    alg_bytes = N * H * W * (C + K) + t * t * K * C
    roof = max(w_ops / (2.0 * peaks["bf16_tflops"] * 1e12), alg_bytes / (peaks["hbm_gbs"] * 1e9))
    return {"layer": name, "N": N, "C": C, "K": K, "H": H, "W": W, "m": m,
            "us": round(us, 2), "path": PATH_NAMES.get(path, str(path)),
            "effective_TOPS": round(d_ops / (us * 1e-6) / 1e12, 1),
            "wino_domain_TOPS": round(w_ops / (us * 1e-6) / 1e12, 1),
            "roofline_us": round(roof * 1e6, 2), "frac": round(roof * 1e6 / us, 4)}


def run_ours(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2002_10711_b200 import binding, cook_toom
    from paper_2002_10711_b200.layer import calibrate

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    # ---- inputs: seeded, synthetic; every rank draws its own batch ----
    wl_r = wi.Workload(**{**wl.__dict__, "seed": wl.seed + 7919 * rank})
    x_q, s_x, w_q, s_w, bias = wi.make_tensors(wl_r)
    BT, G, AT = cook_toom(wl.m)
    if wl.flex:
        BT = wi.flex_perturb(BT, wl.seed, wi.S_BT)
        G = wi.flex_perturb(G, wl.seed, wi.S_G)
        AT = wi.flex_perturb(AT, wl.seed, wi.S_AT)
    q = lambda s, **kw: dict(scale=float(s), **kw)

    def make_plan(s_V, s_U, s_M, s_Y, path=binding.PATH_AUTO):
        return binding.Plan(wl.N, wl.C, wl.H, wl.W, wl.K, wl.m, BT, G, AT, q(s_x), q(s_w), q(s_V),
                            q(s_U), q(s_M), q(s_Y), out_dtype=0, path=path)

    if wl.fixed_scales is not None:
        s_V = s_U = s_M = s_Y = float(np.float32(wl.fixed_scales))
    else:
        s_V, s_U, s_M, s_Y = calibrate(make_plan, x_q, w_q, bias, s_x, s_w, device=dev)
    plan = make_plan(s_V, s_U, s_M, s_Y, path=args.path)

    # ---- device buffers: R rotating sets so that x, y and U_q come from HBM ----
    xb = x_q.nbytes
    yb = wl.N * wl.H * wl.W * wl.K
    R = max(4, int(np.ceil(2 * 126e6 / (xb + yb + plan.weight_bytes))))
    x0 = torch.from_numpy(x_q).to(dev)
    w_dev = torch.from_numpy(w_q).to(dev)
    b_dev = torch.from_numpy(bias).to(dev)
    xs = [x0.clone() for _ in range(R)]
    ys = [torch.empty((wl.N, wl.H, wl.W, wl.K), dtype=torch.int8, device=dev) for _ in range(R)]
    Us = [torch.empty(plan.weight_bytes, dtype=torch.int8, device=dev) for _ in range(R)]
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    for U in Us:
        plan.transform_weights(w_dev, U)
    torch.cuda.synchronize()

    def step(i):
        j = i % R
        plan.conv_forward(xs[j], Us[j], b_dev, ys[j], ws)

    # ---- warm-up (also sets kernel attributes before any capture) ----
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    assert plan.last_status() == 0

    chunk = min(args.steps, 2 * R)
    side = torch.cuda.Stream(device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(chunk):
                step(i)
    torch.cuda.synchronize()
    single_kernel = plan.path in (binding.PATH_SMALLC, binding.PATH_FUSED_F2, binding.PATH_FUSED_LAYER)
    launches_per_step = 1 if single_kernel else 3
    graph.replay()
    torch.cuda.synchronize()

    # ---- timed region ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    replays, rem = divmod(args.steps, chunk)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # spin the clocks up for a moment so the timed region does not start cold
    for _ in range(3):
        graph.replay()
    barrier()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(replays):
        graph.replay()
    for i in range(rem):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    ms_local = e0.elapsed_time(e1)
    status = plan.last_status()
    assert status == 0, binding.strerror(status)
    ms, units = aggregate(ms_local, direct_ops(wl, wl.N) * args.steps, dist if world > 1 else None)
    value = units / (ms * 1e-3) / 1e12
    ms_per_step = ms / args.steps

    # ---- per-kernel times for the roofline: each staged kernel alone, launched
    #      back to back from a CUDA graph on rotating buffers, CUDA events around
    #      the replays (steady-state launch duration, host launch cost excluded) ----
    peaks = load_peaks()
    roofline = None
    stages = None
    if single_kernel:
        # one fused kernel per step: its launch duration is the step time
        alg_bytes = xb + yb + plan.weight_bytes
        ach = alg_bytes / (ms_local / args.steps * 1e-3) / 1e9
        roofline = {"kernel": {binding.PATH_FUSED_F2: "k_fused_f2", binding.PATH_SMALLC: "k_smallc",
                               binding.PATH_FUSED_LAYER: "k_layer_fused"}[plan.path],
                    "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"], "traffic": None,
                    "peak_note": f"of {peaks['source']}"}
    else:
        names = ["input_transform", "hadamard_gemm", "output_transform"]
        us = []
        for mask in (1, 2, 4):
            def stage_step(i, mask=mask):
                j = i % R
                plan.debug_run_stages(mask, xs[j], Us[j], b_dev, ys[j], ws)
            for i in range(3):
                stage_step(i)
            torch.cuda.synchronize()
            sg = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(sg, stream=side):
                    for i in range(2 * R):
                        stage_step(i)
            torch.cuda.synchronize()
            sg.replay()
            torch.cuda.synchronize()
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            nrep = 10
            s0.record()
            for _ in range(nrep):
                sg.replay()
            s1.record()
            torch.cuda.synchronize()
            us.append(s0.elapsed_time(s1) * 1e3 / (nrep * 2 * R))
        # restore the workspace contents of a complete step
        step(0)
        torch.cuda.synchronize()
        t = wl.m + 2
        T = plan.T
        vq = t * t * T * wl.C
        mq = t * t * T * wl.K
        alg = {"input_transform": xb + vq, "hadamard_gemm": vq + plan.weight_bytes + mq,
               "output_transform": mq + yb}
        stages = {n: {"us": u, "algorithmic_bytes": alg[n], "GBps": alg[n] / (u * 1e-6) / 1e9}
                  for n, u in zip(names, us)}
        stages["hadamard_gemm"]["wino_TOPS"] = wino_ops(wl, wl.N) / (us[1] * 1e-6) / 1e12
        dom = max(range(3), key=lambda k: us[k])
        mma_tr = plan.path == binding.PATH_STAGED_TC_MMA
        counters = load_counters() if wl.name == "cfg3" else {}
        # the GEMM of the common configuration runs the lean build of the kernel
        gemm_kernel = "k_gemm_tc_lean" if ("k_gemm_tc_lean" in counters or not counters) else "k_gemm_tc"
        kernel_names = {"input_transform": "k_input_transform_mma" if mma_tr else "k_input_transform_tma",
                        "hadamard_gemm": gemm_kernel,
                        "output_transform": "k_output_transform_mma" if mma_tr else "k_output_transform_tma"}
        traffic_of = lambda k: (counters.get(k) or {}).get("dram_bytes")
        if dom == 1:
            peak = 2.0 * peaks["bf16_tflops"]
            ach = wino_ops(wl, wl.N) / (us[1] * 1e-6) / 1e12
            roofline = {"kernel": gemm_kernel, "bound": "tensor", "achieved": ach, "peak": peak,
                        "unit": "TOP/s", "frac": ach / peak,
                        "traffic": traffic_of(gemm_kernel),
                        "peak_note": f"int8 = 2 x {peaks['source']} bf16 burst peak"}
        else:
            n = names[dom]
            ach = alg[n] / (us[dom] * 1e-6) / 1e9
            roofline = {"kernel": kernel_names[n], "bound": "hbm", "achieved": ach,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                        "traffic": traffic_of(kernel_names[n]),
                        "peak_note": f"of {peaks['source']}"}
    # measured int8 tensor rate of this device: an MMA-only probe kernel (operands in
    # shared memory, accumulators in tensor memory), timed with CUDA events
    mma_probe = None
    if rank == 0:
        iters = 20000
        plan.debug_mma_probe(200)
        torch.cuda.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        plan.debug_mma_probe(iters)
        p1.record()
        torch.cuda.synchronize()
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        mma_probe = sms * iters * 2.0 * 128 * 256 * 32 / (p0.elapsed_time(p1) * 1e-3) / 1e12
        if roofline is not None and roofline["bound"] == "tensor":
            roofline["frac_of_measured_int8_mma"] = roofline["achieved"] / mma_probe
    # whole-layer roofline of the path's definition: slower of MMA work at the int8
    # tensor peak and algorithmic bytes (x + y + U_q) at the HBM peak
    t_mma = wino_ops(wl, wl.N) / (2.0 * peaks["bf16_tflops"] * 1e12)
    t_hbm = (xb + yb + plan.weight_bytes) / (peaks["hbm_gbs"] * 1e9)
    layer_roof = {"t_mma_us": t_mma * 1e6, "t_hbm_us": t_hbm * 1e6,
                  "roofline_us": max(t_mma, t_hbm) * 1e6,
                  "frac": max(t_mma, t_hbm) / (ms_local / args.steps * 1e-3),
                  "peaks": peaks["source"]}
    # third term, which the two-term definition leaves out: plain instruction issue.  Warp
    # instructions per step (ncu smsp__inst_executed.sum, profiles/traffic.json) over
    # SMs x 4 schedulers x 1 instruction per cycle at the maximum SM clock.
    if wl.name == "cfg3" and not single_kernel:
        cnt = load_counters()
        inst = [(cnt.get(k) or {}).get("inst_executed") for k in kernel_names.values()]
        if all(v is not None for v in inst):
            sms = torch.cuda.get_device_properties(dev).multi_processor_count
            t_issue = sum(inst) / (sms * 4 * 1.965e9)
            layer_roof["three_term"] = {
                "warp_instructions_per_step": int(sum(inst)), "t_issue_us": t_issue * 1e6,
                "roofline_us": max(t_mma, t_hbm, t_issue) * 1e6,
                "frac": max(t_mma, t_hbm, t_issue) / (ms_local / args.steps * 1e-3)}

    # ---- the same steps with every buffer resident in L2 (one buffer set): warm-L2 figure ----
    wg_ = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(wg_, stream=side):
            for i in range(chunk):
                plan.conv_forward(xs[0], Us[0], b_dev, ys[0], ws)
    torch.cuda.synchronize()
    wg_.replay()
    torch.cuda.synchronize()
    w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0.record()
    for _ in range(10):
        wg_.replay()
    w1.record()
    torch.cuda.synchronize()
    warm_us = w0.elapsed_time(w1) * 1e3 / (10 * chunk)
    # restore the workspace contents of a complete rotating step
    step(0)
    torch.cuda.synchronize()

    # ---- the single-launch layer kernel on the same workload (extra, not the headline
    #      unless the plan chose it) ----
    single_launch = None
    if rank == 0 and plan.path != binding.PATH_FUSED_LAYER:
        try:
            plan_f = make_plan(s_V, s_U, s_M, s_Y, path=binding.PATH_FUSED_LAYER)
        except binding.WinoError:
            plan_f = None
        if plan_f is not None:
            def fstep(i):
                j = i % R
                plan_f.conv_forward(xs[j], Us[j], b_dev, ys[j], ws)
            for i in range(3):
                fstep(i)
            torch.cuda.synchronize()
            fg = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(fg, stream=side):
                    for i in range(chunk):
                        fstep(i)
            torch.cuda.synchronize()
            fg.replay()
            torch.cuda.synchronize()
            f0_, f1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0_.record()
            for _ in range(10):
                fg.replay()
            f1_.record()
            torch.cuda.synchronize()
            fus = f0_.elapsed_time(f1_) * 1e3 / (10 * chunk)
            single_launch = {"kernel": "k_layer_fused", "us": fus, "launches_per_step": 1,
                             "value": direct_ops(wl, wl.N) / (fus * 1e-6) / 1e12, "unit": UNIT,
                             "frac": max(t_mma, t_hbm) * 1e6 / fus, "status": plan_f.last_status()}
            step(0)
            torch.cuda.synchronize()

    # ---- extra, not the headline: two independent steps in flight on two streams
    #      (each with its own plan and workspace), as a serving loop would run them ----
    overlapped = None
    if not single_kernel:
        plan_b = make_plan(s_V, s_U, s_M, s_Y)
        ws_b = torch.empty(plan_b.workspace_bytes, dtype=torch.uint8, device=dev)
        lanes = [(plan, ws, torch.cuda.Stream(device=dev)), (plan_b, ws_b, torch.cuda.Stream(device=dev))]

        def two_lane(nsteps):
            fork = torch.cuda.Event()
            fork.record(side)
            for _, _, st in lanes:
                st.wait_event(fork)
            for i in range(nsteps):
                pl, w_, st = lanes[i % 2]
                j = i % R
                pl.conv_forward(xs[j], Us[j], b_dev, ys[j], w_, stream=st)
            for _, _, st in lanes:
                join = torch.cuda.Event()
                join.record(st)
                side.wait_event(join)

        with torch.cuda.stream(side):
            two_lane(4)
        torch.cuda.synchronize()
        og = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(og, stream=side):
                two_lane(2 * R)
        torch.cuda.synchronize()
        og.replay()
        torch.cuda.synchronize()
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        o0.record()
        for _ in range(10):
            og.replay()
        o1.record()
        torch.cuda.synchronize()
        o_ms = o0.elapsed_time(o1) / (10 * 2 * R)
        overlapped = {"streams": 2, "ms_per_step": o_ms,
                      "value": direct_ops(wl, wl.N) / (o_ms * 1e-3) / 1e12, "unit": UNIT,
                      "status": plan_b.last_status()}

    # ---- weight transform, timed alone (graph of back-to-back launches) ----
    wg = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(wg, stream=side):
            for i in range(R):
                plan.transform_weights(w_dev, Us[i], stream=side)
    torch.cuda.synchronize()
    wg.replay()
    torch.cuda.synchronize()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(5):
        wg.replay()
    f1.record()
    torch.cuda.synchronize()
    wt_us = f0.elapsed_time(f1) * 1e3 / (5 * R)
    wt_bytes = w_q.nbytes + plan.weight_bytes

    # ---- end to end: pinned host input -> device -> forward -> pinned host output,
    #      every step, through the same C-ABI call; the copies of neighbouring steps
    #      overlap the compute on their own streams (uploads, compute, downloads) ----
    nh = 4
    xh = [torch.from_numpy(x_q).pin_memory() for _ in range(nh)]
    yh = [torch.empty((wl.N, wl.H, wl.W, wl.K), dtype=torch.int8).pin_memory() for _ in range(nh)]
    ke = min(args.steps, 400)
    st_up, st_run, st_down = (torch.cuda.Stream(device=dev) for _ in range(3))

    def e2e_loop(nsteps):
        done_down = [None] * nh
        for i in range(nsteps):
            j, hbuf = i % R, i % nh
            with torch.cuda.stream(st_up):
                xs[j].copy_(xh[hbuf], non_blocking=True)
                up = torch.cuda.Event()
                up.record(st_up)
            st_run.wait_event(up)
            plan.conv_forward(xs[j], Us[j], b_dev, ys[j], ws, stream=st_run)
            ran = torch.cuda.Event()
            ran.record(st_run)
            st_down.wait_event(ran)
            with torch.cuda.stream(st_down):
                yh[hbuf].copy_(ys[j], non_blocking=True)
                done_down[hbuf] = torch.cuda.Event()
                done_down[hbuf].record(st_down)

    # captured as a graph (copy and kernel nodes on three forked streams) so that the
    # host's launch cost does not sit between the copies
    chunk_e = 2 * R
    cur = torch.cuda.current_stream()
    for st in (st_up, st_run, st_down):
        st.wait_stream(cur)
    e2e_loop(8)
    torch.cuda.synchronize()
    eg = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(eg, stream=side):
            for st in (st_up, st_run, st_down):
                st.wait_stream(side)
            e2e_loop(chunk_e)
            for st in (st_up, st_run, st_down):
                side.wait_stream(st)
    torch.cuda.synchronize()
    eg.replay()
    torch.cuda.synchronize()
    reps_e = max(1, ke // chunk_e)
    ke = reps_e * chunk_e
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(reps_e):
        eg.replay()
    g1.record()
    torch.cuda.synchronize()
    barrier()
    assert plan.last_status() == 0
    e2e_ms, e2e_units = aggregate(g0.elapsed_time(g1), direct_ops(wl, wl.N) * ke,
                                  dist if world > 1 else None)
    clocks = sampler.stop() if rank == 0 else None

    # ---- the other configurations (timing only; parity is the GPU tests' job) ----
    other = None
    if rank == 0 and world == 1 and not args.no_other_configs:
        other = []
        for name in ("cfg2", "cfg4"):
            if name == wl.name:
                continue
            o = wi.CONFIGS[name]
            us, pth = time_layer_quick(binding, cook_toom, torch, dev, o.N, o.C, o.H, o.W, o.K, o.m,
                                       flex_seed=o.seed if o.flex else None)
            if us is not None:
                other.append(layer_row(peaks, name, o.N, o.C, o.H, o.W, o.K, o.m, us, pth))
        # the headline layer with per-output-channel scales (staged path, pointer-based
        # output transform)
        us, pth = time_layer_quick(binding, cook_toom, torch, dev, wl.N, wl.C, wl.H, wl.W, wl.K, wl.m,
                                   channel_scales=True)
        if us is not None:
            other.append(layer_row(peaks, wl.name + ".per_channel_scales", wl.N, wl.C, wl.H, wl.W,
                                   wl.K, wl.m, us, pth))
        for ly in wi.resnet18_layers(1005, 256):
            if ly["m"] == 0:
                continue      # stride-2 layers are direct convolutions, not timed
            us, pth = time_layer_quick(binding, cook_toom, torch, dev, ly["N"], ly["C"], ly["H"],
                                       ly["W"], ly["K"], ly["m"])
            if us is not None:
                other.append(layer_row(peaks, f"cfg5.conv{ly['index']}", ly["N"], ly["C"], ly["H"],
                                       ly["W"], ly["K"], ly["m"], us, pth))
        torch.cuda.empty_cache()

    # ---- the oracle beside it (rank 0, single GPU runs only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        import oracle
        L = oracle.Layer(wl.N, wl.C, wl.H, wl.W, wl.K, wl.m, BT, G, AT)
        for qq, s in zip((L.q_x, L.q_w, L.q_V, L.q_U, L.q_M, L.q_Y), (s_x, s_w, s_V, s_U, s_M, s_Y)):
            qq.scale = float(s)
        Uq_ref = oracle.weight_stage(L, w_q)
        y_ref = oracle.forward(L, x_q, U_q=Uq_ref, bias=bias)
        parity = bool((ys[0].cpu().numpy() == y_ref).all()) if rank == 0 else None
        nrun = 5
        t0 = time.perf_counter()
        for _ in range(nrun):
            oracle.forward(L, x_q, U_q=Uq_ref, bias=bias)
        dt = (time.perf_counter() - t0) / nrun
        cpu = {"value": direct_ops(wl, wl.N) / dt / 1e12, "unit": UNIT,
               "cores": oracle.num_threads(), "kind": "oracle",
               "sample": f"full batch N={wl.N}, mean of {nrun} runs ({dt * 1e3:.0f} ms each)",
               "parity_with_gpu_output": parity}

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": workload_config(
                wl, f"inputs rotate over {R} buffer sets ({R * (xb + yb + plan.weight_bytes) / 1e6:.0f} MB > L2)"),
            "wino_domain_TOPS": wino_ops(wl, wl.N) * world / (ms_per_step * 1e-3) / 1e12,
            "path": PATH_NAMES[plan.path],
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "layer_roofline": layer_roof, "stages": stages,
            "warm_l2": {"ms_per_step": warm_us * 1e-3,
                        "value": direct_ops(wl, wl.N) / (warm_us * 1e-6) / 1e12, "unit": UNIT,
                        "note": "every step on one buffer set (x, U_q, y stay in L2)"},
            "single_launch": single_launch, "other_configs": other,
            "int8_mma_probe_TOPS": mma_probe,
            "weight_transform": {"us": wt_us, "GBps": wt_bytes / (wt_us * 1e-6) / 1e9,
                                 "algorithmic_bytes": wt_bytes},
            "overlapped_steps": overlapped,
            "e2e": {"value": e2e_units / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": xb, "d2h_bytes_per_step": yb, "steps": ke},
            "cpu_baseline": cpu, "clocks": clocks,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=sorted(wi.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the timing rows of cfg2, cfg4 and the cfg5 layers")
    ap.add_argument("--path", type=int, default=0,
                    help="pin the execution path (WINO_PATH_* number; 0 = the plan's own choice)")
    args = ap.parse_args()
    wl = wi.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
