"""Property tier: seeded random layer shapes, tile sizes, matrices (Cook-Toom or
perturbed), quantizer options and execution paths; every case must match the
oracle byte for byte (float outputs within 1e-4 of the output's max magnitude)."""
import numpy as np
import pytest

import oracle
import wino_inputs as wi
from helpers import build_layer, per_channel

pytestmark = pytest.mark.gpu


def _cases(n, seed):
    draws = wi.bits64(seed, 99, 16 * n).reshape(n, 16)
    out = []
    for d in draws:
        pick = lambda i, opts: opts[int(d[i] % np.uint64(len(opts)))]
        m = pick(0, [2, 4, 6])
        C = pick(1, [4, 8, 16, 20, 32, 48, 64, 96, 128, 160, 256])
        K = pick(2, [4, 12, 16, 32, 48, 64, 80, 128, 192, 256, 272])
        H = 1 + int(d[3] % np.uint64(14))
        W = 1 + int(d[4] % np.uint64(14))
        N = 1 + int(d[5] % np.uint64(6))
        out.append(dict(m=m, C=C, K=K, H=H, W=W, N=N, flex=bool(d[6] & np.uint64(1)),
                        q_M=bool(d[7] % np.uint64(4)), out_dtype=int(d[8] % np.uint64(4) == 0),
                        relu=bool(d[9] & np.uint64(1)), with_bias=bool(d[10] % np.uint64(3)),
                        zp=bool(d[11] % np.uint64(4) == 0), path_draw=int(d[12] % np.uint64(97)),
                        seed=int(d[13] % np.uint64(100000)),
                        per_channel=bool(d[14] % np.uint64(3) == 0)))
    return out


def check_case(case):
    from gpu_helpers import gpu_run
    from paper_2002_10711_b200 import binding
    wl = wi.Workload("r", case["seed"], case["N"], case["C"], case["H"], case["W"], case["K"], case["m"],
                     flex=case["flex"])
    L, x_q, w_q, bias = build_layer(wl, q_M=case["q_M"], out_dtype=case["out_dtype"], relu=case["relu"],
                                    with_bias=case["with_bias"])
    if case["zp"]:
        L.q_x.zero_point, L.q_w.zero_point, L.q_Y.zero_point = 3, -2, 5
    if case["per_channel"]:
        L = per_channel(L, case["seed"] + 1, spread=3.0)
    supported = []
    # per-channel scales exist on the staged paths; a plan forced elsewhere moves to one
    for path in ((1, 2, 4) if case["per_channel"] else (1, 2, 3, 4, 5, 6, 7)):
        try:
            binding.Plan.from_layer(L, path=path)
            supported.append(path)
        except binding.WinoError as e:
            assert e.code == binding.ERR_UNSUPPORTED
    assert supported
    path = supported[case["path_draw"] % len(supported)]
    y_ref = oracle.forward(L, x_q, w_q, bias=bias)
    g = gpu_run(L, x_q, w_q, bias, path=path)
    assert g["path"] == path
    if L.out_dtype == 0:
        assert (g["y"] == y_ref).all(), (case, path)
    else:
        tol = 1e-4 * max(float(np.abs(y_ref).max()), 1e-30)
        assert float(np.abs(g["y"] - y_ref).max()) <= tol, (case, path)
    # the automatic choice must agree as well
    g2 = gpu_run(L, x_q, w_q, bias)
    if L.out_dtype == 0:
        assert (g2["y"] == y_ref).all(), (case, "auto", g2["path"])


@pytest.mark.parametrize("case", _cases(64, 20260), ids=lambda c: f"m{c['m']}C{c['C']}K{c['K']}H{c['H']}W{c['W']}")
def test_random_layer(case):
    check_case(case)
