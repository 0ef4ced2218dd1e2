"""CPU-side checks of the CUDA library: it loads, exports every symbol the
header declares, and its host logic (validation, sizes, path choice,
multipliers) behaves.  No kernel runs here."""
import ctypes as ct
import os
import re

import numpy as np
import pytest

import oracle
import wino_inputs as wi
from paper_2002_10711_b200 import binding, cook_toom, cook_toom_exact
from paper_2002_10711_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _plan(N=2, C=64, H=8, W=8, K=64, m=4, **kw):
    BT, G, AT = cook_toom(m)
    q = dict(scale=0.1)
    args = dict(q_x=q, q_w=q, q_V=q, q_U=q, q_M=q, q_Y=q)
    args.update(kw)
    return binding.Plan(N, C, H, W, K, m, BT, G, AT, **args)


def test_library_builds_and_exports_header_symbols():
    lib = ct.CDLL(build())
    header = open(os.path.join(ROOT, "include", "wino.h")).read()
    declared = set(re.findall(r"\b(wino_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("m", [2, 4, 6])
def test_product_matrices_match_oracle_construction(m):
    mine = cook_toom(m)
    ref = oracle.cook_toom(m, wi.POINTS[m])
    for a, k in zip(mine, ("BT32", "G32", "AT32")):
        assert (a.view(np.uint32) == ref[k].view(np.uint32)).all()
    ex = cook_toom_exact(m)
    for a, k in zip(ex, ("BT", "G", "AT")):
        assert (np.array(a, dtype=object) == ref[k]).all()


def test_sizes_and_paths():
    p = _plan()
    assert p.weight_bytes == 36 * 64 * 64
    assert p.T == 2 * 2 * 2
    assert p.workspace_bytes >= 36 * p.T * 64 * 2
    assert p.path == binding.PATH_STAGED_TC
    assert _plan(C=16, K=16).path == binding.PATH_STAGED_DP4A     # at most 16 channels: integer dot products
    assert _plan(C=32, K=16).path == binding.PATH_STAGED_TC
    assert _plan(C=20, K=24).path == binding.PATH_STAGED_DP4A
    p = _plan(C=20, K=24)
    p.force_path(binding.PATH_SMALLC)
    assert p.path == binding.PATH_SMALLC
    assert _plan(C=36, K=40).path == binding.PATH_STAGED_DP4A
    assert _plan(m=2, C=64, K=64).path == binding.PATH_FUSED_F2
    assert _plan(m=2, C=64, K=128).path == binding.PATH_STAGED_TC
    p = _plan(C=64, K=64)
    p.force_path(binding.PATH_STAGED_DP4A)
    assert p.path == binding.PATH_STAGED_DP4A
    with pytest.raises(binding.WinoError) as e:
        p.force_path(binding.PATH_SMALLC)
    assert e.value.code == binding.ERR_UNSUPPORTED
    # Q_M disabled: the middle buffer holds int32
    q = dict(scale=0.1)
    assert _plan(q_M=dict(scale=0.1, enabled=0)).workspace_bytes > _plan().workspace_bytes


def test_validation_errors():
    for kw, code in ((dict(m=3), binding.ERR_UNSUPPORTED), (dict(C=3), binding.ERR_UNSUPPORTED),
                     (dict(N=0), binding.ERR_INVALID), (dict(C=2048), binding.ERR_UNSUPPORTED),
                     (dict(q_V=dict(scale=0.1, zero_point=3)), binding.ERR_UNSUPPORTED),
                     (dict(q_x=dict(scale=-1.0)), binding.ERR_INVALID),
                     (dict(q_Y=dict(scale=0.1, qmin=-300)), binding.ERR_INVALID),
                     (dict(out_dtype=5), binding.ERR_INVALID)):
        with pytest.raises(binding.WinoError) as e:
            if "m" in kw:
                BT, G, AT = cook_toom(4)
                q = dict(scale=0.1)
                binding.Plan(1, 16, 8, 8, 16, 3, BT, G, AT, q, q, q, q, q, q)
            else:
                _plan(**kw)
        assert e.value.code == code, kw
    BT, G, AT = cook_toom(4)
    BT = BT.copy(); BT[0, 0] = np.nan
    q = dict(scale=0.1)
    with pytest.raises(binding.WinoError):
        binding.Plan(1, 16, 8, 8, 16, 4, BT, G, AT, q, q, q, q, q, q)


def test_multipliers_match_oracle_definition():
    ct_ = oracle.cook_toom(4, wi.POINTS[4])
    L = oracle.Layer(1, 16, 8, 8, 16, 4, ct_["BT32"], ct_["G32"], ct_["AT32"])
    for q, s in zip((L.q_x, L.q_w, L.q_V, L.q_U, L.q_M, L.q_Y), (0.031, 0.0017, 0.093, 0.0009, 0.011, 0.047)):
        q.scale = s
    for en in (1, 0):
        L.q_M.enabled = en
        p = binding.Plan.from_layer(L)
        assert (p.multipliers().view(np.uint32) == oracle.multipliers(L).view(np.uint32)).all()


def test_null_and_alignment_checks_without_gpu():
    p = _plan()
    lib = binding._lib
    assert lib.wino_conv_forward(p._h, None, None, None, None, None, None) == binding.ERR_INVALID
    assert lib.wino_conv_forward(p._h, 17, 32, None, 48, 64, None) == binding.ERR_ALIGNMENT
    assert lib.wino_transform_weights(p._h, 16, 33, None, None) == binding.ERR_ALIGNMENT
    assert lib.wino_debug_dump_stage(p._h, 0, 16, 10) == binding.ERR_UNSUPPORTED  # no forward yet
    assert binding.strerror(binding.ERR_TIMEOUT).startswith("bounded")


def test_once_per_device_bookkeeping():
    # kernel attributes are set once on every device a kernel runs on: the table is keyed
    # by device index, so a second device gets its own first time
    assert binding.debug_once_per_device(3) == 1
    assert binding.debug_once_per_device(3) == 0
    assert binding.debug_once_per_device(4) == 1
    assert binding.debug_once_per_device(3) == 0
    assert binding.debug_once_per_device(63) == 1
    assert binding.debug_once_per_device(64) == binding.ERR_INVALID
    assert binding.debug_once_per_device(-1) == binding.ERR_INVALID


def test_channel_scales_are_validated_on_the_host():
    p = _plan(C=64, K=64, m=2)            # a layer the fused F2 kernel would take
    ok = np.full(64, 0.1, np.float32)
    bad = ok.copy(); bad[7] = 0.0
    nan = ok.copy(); nan[3] = np.nan
    lib = binding._lib
    for arr in (bad, nan, -ok):
        assert lib.wino_plan_set_channel_scales(p._h, arr.ctypes.data, None, None, None) == binding.ERR_INVALID
        assert lib.wino_plan_set_channel_scales(p._h, None, None, arr.ctypes.data, None) == binding.ERR_INVALID
        assert lib.wino_plan_set_channel_scales(p._h, None, None, None, arr.ctypes.data) == binding.ERR_INVALID
    before = p.path
    assert lib.wino_plan_set_channel_scales(p._h, None, None, None, None) == binding.WINO_OK   # nothing to undo
    assert p.path == before
    with pytest.raises(ValueError):
        p.set_channel_scales(np.ones(3, np.float32))
    rc = lib.wino_plan_set_channel_scales(p._h, ok.ctypes.data, None, None, None)
    assert rc in (binding.WINO_OK, binding.ERR_CUDA)      # needs a device for its table
    if rc == binding.WINO_OK:
        assert p.path == binding.PATH_STAGED_TC
