"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle, element by element on the same seeded inputs.  Integer stages (the int32
Hadamard sums on every path, single-kernel paths included) and int8 outputs
must be bit-exact.  Float outputs must meet the stated tolerance of 1e-4 of the
output's max magnitude; because both sides execute the same fused-multiply-add
chains in the same order they are also required to be identical."""
import numpy as np
import pytest

import oracle
import wino_inputs as wi
from helpers import build_layer, per_channel, small

pytestmark = pytest.mark.gpu

TC, DP4A, SMALLC, TC_PTR, FUSED, TC_MMA, LAYER = 1, 2, 3, 4, 5, 6, 7


def _compare(L, x_q, w_q, bias, path, dumps=True):
    from gpu_helpers import gpu_run
    y_ref, d_ref = oracle.forward(L, x_q, w_q, bias=bias, dumps=True)
    g = gpu_run(L, x_q, w_q, bias, path=path, dumps=dumps)
    assert g["path"] == path
    assert (g["U_q"] == d_ref["U_q"]).all(), "U_q"
    if "M" in g:   # staged paths with dumps, and the single-kernel paths always
        assert (g["M"] == d_ref["M"]).all(), "M"
    if dumps:
        assert (g["V_q"] == d_ref["V_q"]).all(), "V_q"
        if L.q_M.enabled:
            assert (g["m_q"] == d_ref["m_q"]).all(), "m_q"
    if L.out_dtype == 0:
        bad = np.count_nonzero(g["y"] != y_ref)
        assert bad == 0, f"y differs in {bad} of {y_ref.size}"
    else:
        tol = 1e-4 * max(float(np.abs(y_ref).max()), 1e-30)
        assert float(np.abs(g["y"] - y_ref).max()) <= tol
        bad = np.count_nonzero(g["y"].view(np.uint32) != y_ref.view(np.uint32))
        assert bad == 0, f"float y differs in {bad} of {y_ref.size}"
    return g


SHAPES = [
    # N, C, H, W, K
    (1, 16, 8, 8, 16),
    (2, 32, 7, 9, 48),       # ragged tiles, K not a multiple of 32
    (3, 64, 13, 5, 64),
    (1, 160, 6, 6, 80),      # C spans two 128-byte stages with a partial one
    (5, 48, 10, 11, 272),    # K > 256: two column blocks
    (2, 128, 9, 10, 192),    # TMA-staged transforms: 128- and 64-channel chunks, ragged tiles
    (1, 512, 4, 4, 512),     # 256-channel chunks, two per tile
    (3, 256, 7, 7, 128),     # odd tile count: last block of a 2-tile group is partial
    (37, 128, 9, 9, 256),    # tensor-core transforms: more units than resident blocks, ragged tiles
    (4, 384, 8, 8, 384),     # three 128-channel stages; the second 256-wide column block is half empty
]


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("path", [TC, TC_MMA, TC_PTR, DP4A])
def test_staged_paths_every_stage(m, shape, path):
    N, C, H, W, K = shape
    wl = wi.Workload("s", 3000 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    _compare(L, x_q, w_q, bias, path)


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("path", [TC, DP4A, SMALLC])
def test_flex_matrices(m, path):
    C = 32 if path == SMALLC else 64
    wl = wi.Workload("f", 3100 + m, 2, C, 9, 7, C, m, flex=True)
    L, x_q, w_q, bias = build_layer(wl)
    _compare(L, x_q, w_q, bias, path, dumps=path != SMALLC)


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("path", [TC, TC_PTR, DP4A, SMALLC])
@pytest.mark.parametrize("variant", ["no_qm", "float_out", "no_qm_float", "relu", "no_bias", "zero_points"])
def test_variants(m, path, variant):
    C, K = (16, 32) if path == SMALLC else (64, 64)
    wl = wi.Workload("v", 3200 + m, 2, C, 8, 10, K, m)
    kw = {}
    if variant in ("no_qm", "no_qm_float"):
        kw["q_M"] = False
    if variant in ("float_out", "no_qm_float"):
        kw["out_dtype"] = 1
    if variant == "relu":
        kw["relu"] = True
    if variant == "no_bias":
        kw["with_bias"] = False
    L, x_q, w_q, bias = build_layer(wl, **kw)
    if variant == "zero_points":
        L.q_x.zero_point = 5
        L.q_w.zero_point = -3
        L.q_Y.zero_point = 7
    _compare(L, x_q, w_q, bias, path, dumps=path != SMALLC)


@pytest.mark.parametrize("shape", [(1, 4, 3, 3, 4), (2, 8, 1, 1, 12), (1, 32, 5, 20, 32), (7, 20, 6, 6, 28)])
@pytest.mark.parametrize("m", [2, 4, 6])
def test_small_channel_path(m, shape):
    N, C, H, W, K = shape
    wl = wi.Workload("c", 3300 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    _compare(L, x_q, w_q, bias, SMALLC, dumps=False)
    _compare(L, x_q, w_q, bias, DP4A, dumps=True)


LAYER_SHAPES = [
    # N, C, H, W, K  (C and K multiples of 128)
    (1, 128, 8, 8, 128),      # a handful of tiles: most CTAs have nothing to do
    (2, 128, 9, 10, 256),     # ragged tiles
    (37, 128, 9, 9, 256),     # several 128-tile blocks, the last one partial
    (1, 512, 4, 4, 512),      # four channel chunks, two 256-wide column blocks
    (3, 256, 7, 7, 128),
    (16, 384, 8, 8, 384),     # second column block half empty
    (60, 128, 16, 16, 128),   # many blocks of tiles: every CTA loops in all three phases
]


@pytest.mark.parametrize("m", [2, 4])
@pytest.mark.parametrize("shape", LAYER_SHAPES)
def test_single_launch_layer_every_stage(m, shape):
    N, C, H, W, K = shape
    wl = wi.Workload("l", 3900 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    g = _compare(L, x_q, w_q, bias, LAYER)
    assert g["launches"] == 2          # weight transform + one launch for the whole layer


@pytest.mark.parametrize("variant", ["relu", "no_bias", "zero_points_w_y", "saturating"])
def test_single_launch_layer_variants(variant):
    wl = wi.Workload("lv", 3950, 5, 256, 8, 10, 128, 4)
    kw = {}
    if variant == "relu":
        kw["relu"] = True
    if variant == "no_bias":
        kw["with_bias"] = False
    L, x_q, w_q, bias = build_layer(wl, **kw)
    if variant == "zero_points_w_y":
        L.q_w.zero_point = -3
        L.q_Y.zero_point = 7
    if variant == "saturating":
        for q in (L.q_V, L.q_U, L.q_M, L.q_Y):
            q.scale = q.scale / 7.0
    _compare(L, x_q, w_q, bias, LAYER)


def test_single_launch_layer_back_to_back_calls_reuse_the_counters():
    import torch
    from paper_2002_10711_b200 import binding
    from paper_2002_10711_b200.layer import WinogradConv
    wl = wi.Workload("lb", 3960, 9, 128, 8, 8, 256, 4)
    L, x_q, w_q, bias = build_layer(wl)
    y_ref = oracle.forward(L, x_q, w_q, bias=bias)
    plan = binding.Plan.from_layer(L, path=LAYER)
    conv = WinogradConv(plan)
    conv.load_weights(w_q, bias)
    x = torch.from_numpy(x_q).cuda()
    ys = [conv.forward(x, conv.empty_output().fill_(0)) for _ in range(5)]
    assert plan.last_status() == 0
    for y in ys:
        assert (y.cpu().numpy() == y_ref).all()


def test_single_launch_layer_refuses_other_layers():
    from paper_2002_10711_b200 import binding
    for m, C, K, flex, kw in ((6, 128, 128, False, {}), (4, 64, 128, False, {}), (4, 128, 192, False, {}),
                              (4, 128, 128, True, {}), (4, 128, 128, False, {"out_dtype": 1}),
                              (4, 128, 128, False, {"q_M": False})):
        wl = wi.Workload("lr", 3970, 1, C, 8, 8, K, m, flex=flex)
        L, x_q, w_q, bias = build_layer(wl, **kw)
        with pytest.raises(binding.WinoError) as e:
            binding.Plan.from_layer(L, path=LAYER)
        assert e.value.code == binding.ERR_UNSUPPORTED


FUSED_SHAPES = [
    # N, C, H, W, K
    (2, 64, 8, 8, 64),
    (1, 32, 7, 9, 48),        # ragged tiles; K = 48: second 32-channel block half empty
    (3, 64, 13, 5, 16),
    (1, 32, 32, 32, 32),
    (40, 64, 32, 32, 64),     # 10240 tiles = 80 blocks of 128
    (100, 64, 30, 30, 64),    # 22500 tiles: more blocks than SMs, last block partial
]


@pytest.mark.parametrize("shape", FUSED_SHAPES)
def test_fused_f2_kernel(shape):
    N, C, H, W, K = shape
    wl = wi.Workload("fu", 3500 + C + K, N, C, H, W, K, 2)
    L, x_q, w_q, bias = build_layer(wl)
    from paper_2002_10711_b200 import binding
    assert binding.Plan.from_layer(L).path == FUSED      # the automatic choice for these shapes
    _compare(L, x_q, w_q, bias, FUSED, dumps=False)


@pytest.mark.parametrize("variant", ["no_qm", "float_out", "no_qm_float", "relu", "no_bias", "zero_points"])
def test_fused_f2_variants(variant):
    wl = wi.Workload("fv", 3600, 3, 64, 10, 12, 64, 2)
    kw = {}
    if variant in ("no_qm", "no_qm_float"):
        kw["q_M"] = False
    if variant in ("float_out", "no_qm_float"):
        kw["out_dtype"] = 1
    if variant == "relu":
        kw["relu"] = True
    if variant == "no_bias":
        kw["with_bias"] = False
    L, x_q, w_q, bias = build_layer(wl, **kw)
    if variant == "zero_points":
        L.q_x.zero_point = 5
        L.q_w.zero_point = -3
        L.q_Y.zero_point = 7
    _compare(L, x_q, w_q, bias, FUSED, dumps=False)


def test_fused_f2_refuses_other_shapes():
    from paper_2002_10711_b200 import binding
    for m, C, K, flex in ((4, 64, 64, False), (2, 128, 64, False), (2, 64, 128, False), (2, 64, 64, True)):
        wl = wi.Workload("fr", 3700, 1, C, 8, 8, K, m, flex=flex)
        L, x_q, w_q, bias = build_layer(wl)
        with pytest.raises(binding.WinoError) as e:
            binding.Plan.from_layer(L, path=FUSED)
        assert e.value.code == binding.ERR_UNSUPPORTED


# ---------------------------------------------------------------------------
# Per-output-channel scales (Section 7) and stage code ranges narrower than eight bits
# (Section 3.2: every intermediate may have its own bit-width).
# ---------------------------------------------------------------------------
PC_SHAPES = [(2, 32, 7, 9, 48), (5, 48, 10, 11, 272), (2, 128, 9, 10, 192), (3, 256, 7, 7, 128)]


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("shape", PC_SHAPES)
@pytest.mark.parametrize("path", [TC, TC_PTR, DP4A])
def test_per_channel_scales_every_stage(m, shape, path):
    N, C, H, W, K = shape
    wl = wi.Workload("pc", 4000 + m, N, C, H, W, K, m)
    L, x_q, w_q, bias = build_layer(wl)
    _compare(per_channel(L, 17 + m, spread=3.0), x_q, w_q, bias, path)


@pytest.mark.parametrize("path", [TC, TC_PTR, DP4A])
@pytest.mark.parametrize("variant", ["no_qm", "float_out", "no_qm_float", "relu", "zero_points", "flex"])
def test_per_channel_scales_variants(path, variant):
    wl = wi.Workload("pcv", 4100, 3, 64, 9, 6, 80, 4, flex=(variant == "flex"))
    L, x_q, w_q, bias = build_layer(wl, q_M=not variant.startswith("no_qm"),
                                    out_dtype=1 if "float" in variant else 0,
                                    relu=(variant == "relu"))
    if variant == "zero_points":
        L.q_x.zero_point, L.q_w.zero_point, L.q_Y.zero_point = 3, -2, 5
    _compare(per_channel(L, 23), x_q, w_q, bias, path)


def test_per_channel_scales_move_single_kernel_plans_to_a_staged_path():
    from paper_2002_10711_b200 import binding
    wl = wi.Workload("pcf", 4200, 2, 64, 8, 8, 64, 2)
    L, x_q, w_q, bias = build_layer(wl)
    plan = binding.Plan.from_layer(L)
    assert plan.path == FUSED
    P = per_channel(L, 5)
    plan.set_channel_scales(P.s_w_K, P.s_U_K, P.s_M_K, P.s_Y_K)
    assert plan.path == TC
    for refused in (FUSED, SMALLC, TC_MMA, LAYER):
        with pytest.raises(binding.WinoError):
            plan.force_path(refused)
    plan.set_channel_scales(None, None, None, None)       # back to per-layer scales
    plan.force_path(FUSED)
    with pytest.raises(binding.WinoError):
        plan.set_channel_scales(np.zeros(L.K, np.float32), None, None)
    g = _compare(P, x_q, w_q, bias, TC)
    assert g["launches"] >= 4


def test_only_some_channel_scales_given():
    wl = wi.Workload("pcs", 4300, 2, 32, 6, 6, 32, 4)
    L, x_q, w_q, bias = build_layer(wl)
    P = per_channel(L, 9)
    P.s_U_K = None; P.s_M_K = None                  # weights and output per channel, U and M per layer
    _compare(P, x_q, w_q, bias, TC)
    P = per_channel(L, 10)
    P.s_w_K = None; P.s_Y_K = None
    _compare(P, x_q, w_q, bias, DP4A)
    P = per_channel(L, 11)
    P.s_w_K = None; P.s_U_K = None; P.s_Y_K = None  # only the Hadamard sums per channel
    _compare(P, x_q, w_q, bias, TC_PTR)


@pytest.mark.parametrize("path", [TC, TC_PTR, DP4A])
@pytest.mark.parametrize("m", [2, 4, 6])
def test_narrow_code_ranges_per_stage(path, m):
    """6-bit V, 5-bit U, 7-bit M and a 4-bit output, each with its own calibrated-then-widened
    scale: clamps at every stage, identical codes."""
    wl = wi.Workload("bits", 4400 + m, 3, 48, 9, 7, 64, m)
    L, x_q, w_q, bias = build_layer(wl)
    for q, bits in ((L.q_V, 6), (L.q_U, 5), (L.q_M, 7), (L.q_Y, 4)):
        top = 2 ** (bits - 1) - 1
        q.scale = float(np.float32(q.scale * 127.0 / top * 0.8))   # 0.8: some values clip
        q.qmin, q.qmax = -top, top
    g = _compare(L, x_q, w_q, bias, path)
    assert np.abs(g["V_q"]).max() == 31 and np.abs(g["y"]).max() == 7


def test_saturating_scales_clip_identically():
    wl = wi.Workload("sat", 3400, 2, 32, 8, 8, 32, 4)
    L, x_q, w_q, bias = build_layer(wl)
    for q in (L.q_V, L.q_U, L.q_M, L.q_Y):
        q.scale = q.scale / 7.0           # most values clip
    g = _compare(L, x_q, w_q, bias, TC)
    assert np.abs(g["V_q"]).max() == 127 and (np.abs(g["V_q"]) == 127).mean() > 0.05


# --- the five workload configurations -------------------------------------------------
def test_cfg1_all_paths():
    wl = wi.CONFIGS["cfg1"]
    L, x_q, w_q, bias = build_layer(wl)
    for path in (SMALLC, TC, DP4A):
        _compare(L, x_q, w_q, bias, path, dumps=path != SMALLC)


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4"])
def test_full_size_configs(name):
    wl = wi.CONFIGS[name]
    L, x_q, w_q, bias = build_layer(wl)
    g = _compare(L, x_q, w_q, bias, TC)
    assert g["launches"] >= 4
    _compare(L, x_q, w_q, bias, TC_MMA)
    if name == "cfg3":
        _compare(L, x_q, w_q, bias, LAYER)
    _compare(L, x_q, w_q, bias, TC_PTR)
    if name == "cfg2":
        _compare(L, x_q, w_q, bias, FUSED, dumps=False)


def test_cfg3_without_qm():
    wl = small(wi.CONFIGS["cfg3"], N=32)
    L, x_q, w_q, bias = build_layer(wl, q_M=False)
    _compare(L, x_q, w_q, bias, TC)


def test_gpu_calibration_matches_oracle_calibration():
    from paper_2002_10711_b200 import binding
    from paper_2002_10711_b200.layer import calibrate
    for name, N in (("cfg2", 2), ("cfg3", 8), ("cfg4", 2)):
        wl = small(wi.CONFIGS[name], N=N)
        L, x_q, w_q, bias = build_layer(wl)

        def make_plan(s_V, s_U, s_M, s_Y):
            import copy
            L2 = copy.deepcopy(L)
            L2.q_V.scale, L2.q_U.scale, L2.q_M.scale, L2.q_Y.scale = s_V, s_U, s_M, s_Y
            return binding.Plan.from_layer(L2)

        got = calibrate(make_plan, x_q, w_q, bias, L.q_x.scale, L.q_w.scale)
        want = (L.q_V.scale, L.q_U.scale, L.q_M.scale, L.q_Y.scale)
        assert tuple(np.float32(got)) == tuple(np.float32(want)), (name, got, want)


@pytest.mark.parametrize("m,q_M,per_k_out", [(2, True, False), (4, True, True), (6, False, False)])
def test_gpu_per_channel_calibration_matches_oracle_calibration(m, q_M, per_k_out):
    """The library-side per-channel calibration (per-filter statistic of the weight transform,
    stage dumps) against the oracle's, scale for scale; then the layer under those scales."""
    import copy
    from paper_2002_10711_b200 import binding
    from paper_2002_10711_b200.layer import calibrate_per_channel
    from oracle.calibrate import calibrate_per_channel as oracle_calibrate
    wl = wi.Workload("pccal2", 4600 + m, 3, 32, 9, 7, 48, m)
    L, x_q, w_q, bias = build_layer(wl, q_M=q_M)
    L.s_w_K = (np.float32(L.q_w.scale) * wi.channel_factors(77, L.K, 3.0)[0]).astype(np.float32)
    want = oracle_calibrate(L, x_q, w_q, bias, output_per_channel=per_k_out)

    def make_plan(s_V, s_U, s_M, s_Y, out_dtype):
        L2 = copy.deepcopy(L)
        L2.s_w_K = None
        L2.q_V.scale, L2.q_U.scale, L2.q_M.scale, L2.q_Y.scale = s_V, s_U, s_M, s_Y
        L2.out_dtype = out_dtype
        return binding.Plan.from_layer(L2)

    s_V, s_U_K, s_M_K, s_Y = calibrate_per_channel(make_plan, x_q, w_q, bias, L.q_x.scale, L.s_w_K,
                                                   output_per_channel=per_k_out)
    assert np.float32(s_V) == np.float32(want.q_V.scale)
    assert (s_U_K.view(np.uint32) == want.s_U_K.view(np.uint32)).all()
    if q_M:
        assert (s_M_K.view(np.uint32) == want.s_M_K.view(np.uint32)).all()
    else:
        assert s_M_K is None and want.s_M_K is None
    if per_k_out:
        assert (s_Y.view(np.uint32) == want.s_Y_K.view(np.uint32)).all()
    else:
        assert np.float32(s_Y) == np.float32(want.q_Y.scale)
    g = _compare(want, x_q, w_q, bias, TC)
    assert np.abs(g["y"]).max() >= 120          # the calibrated output scale fills the range


@pytest.mark.parametrize("path", [TC, DP4A])
def test_calibration_statistics_with_channel_scales(path):
    """The four max-abs statistics of a calibration pass on a plan with per-channel scales,
    against the same maxima taken over the oracle's stage outputs."""
    import copy
    import torch
    from paper_2002_10711_b200 import binding
    wl = wi.Workload("pccal", 4500, 3, 64, 9, 7, 80, 4)
    L, x_q, w_q, bias = build_layer(wl)
    P = per_channel(L, 41, spread=3.0)
    plan = binding.Plan.from_layer(P, path=path)
    x = torch.from_numpy(x_q).cuda()
    w = torch.from_numpy(w_q).cuda()
    b = torch.from_numpy(bias).cuda()
    U = torch.empty(plan.weight_bytes, dtype=torch.int8, device="cuda")
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device="cuda")
    stats = torch.zeros(4, dtype=torch.int32, device="cuda")
    plan.transform_weights(w, U)
    plan.calibrate_forward(x, U, b, None, ws, stats)
    assert plan.last_status() == 0
    got = stats.cpu().numpy().view(np.float32)
    _, Vf = oracle.input_stage(P, x_q, want_f32=True)
    _, d = oracle.forward(P, x_q, w_q, bias=bias, dumps=True)
    _, Yf = oracle.output_stage(P, d["M"], d["m_q"], bias, want_f32=True)
    F = copy.deepcopy(P)
    F.out_dtype = 1
    y_float = oracle.forward(F, x_q, w_q, bias=bias)
    want = np.array([np.abs(Vf).max(), np.abs(d["M"]).max(), np.abs(Yf).max(), np.abs(y_float).max()],
                    np.float32)
    assert (got.view(np.uint32) == want.view(np.uint32)).all(), (got, want)


def test_mma_probe_runs_and_reports_ok():
    import torch
    from paper_2002_10711_b200 import binding, cook_toom
    BT, G, AT = cook_toom(4)
    q = dict(scale=0.1)
    plan = binding.Plan(2, 64, 8, 8, 64, 4, BT, G, AT, q, q, q, q, q, q)
    plan.debug_mma_probe(500)
    assert plan.last_status() == 0
    with pytest.raises(binding.WinoError):
        plan.debug_mma_probe(0)


def test_bounded_wait_expires_with_an_error_and_the_plan_stays_usable():
    """A wait nothing satisfies gives up after its cycle limit: the kernel leaves by its
    normal exit, the status word reports the timeout once (read-and-clear), and a
    forward pass afterwards is still bit-exact."""
    from paper_2002_10711_b200 import binding
    wl = wi.Workload("wp", 3800, 2, 64, 8, 8, 64, 4)
    L, x_q, w_q, bias = build_layer(wl)
    plan = binding.Plan.from_layer(L)
    plan.debug_wait_probe(100000)
    assert plan.last_status() == binding.ERR_TIMEOUT
    assert plan.last_status() == 0                  # cleared by the read
    with pytest.raises(binding.WinoError):
        plan.debug_wait_probe(0)
    _compare(L, x_q, w_q, bias, TC)
