"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every symbol the public header declares, and validates arguments."""
import ctypes
import os
import re

import pytest

from paper_2409_12210_b200 import binding as B
from paper_2409_12210_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    libbuild.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "modse.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(modse_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.lib_path())
    names = declared_symbols()
    assert "modse_create" in names and "modse_forward" in names and "modse_backward" in names
    assert "modse_destroy" in names
    for n in names:
        assert getattr(lib, n) is not None, n


def test_create_validation():
    ok = B.ModseLayer(64, [96, 160, 112, 144], 2)
    ok.destroy()
    B.ModseLayer(2048, [5632], 1).destroy()                   # one expert, top-1 is legal
    for args in [(60, [96, 160], 2), (64, [96, 100], 2), (64, [96, 160], 3), (64, [96, 160], 0),
                 (64, [8, 160], 1), (64, [], 1)]:
        with pytest.raises(B.ModseError) as ei:
            B.ModseLayer(*args)
        assert ei.value.status == B.MODSE_ERR_INVALID_ARG
    with pytest.raises(B.ModseError) as ei:
        B.ModseLayer(64, [96, 160, 112, 144], 3)               # legal layer, not run by the CUDA path
    assert ei.value.status == B.MODSE_ERR_UNSUPPORTED
    assert B.load().modse_destroy(None) == B.MODSE_OK


def test_pair_rule_helper():
    assert B.check_pairs([2816, 8448, 3520, 7744, 4224, 7040, 4928, 6336]) == (True, 11264)
    assert B.check_pairs([9216, 1024, 8192, 2048, 6144, 4096, 5120, 5120]) == (True, 10240)   # Table 2
    assert B.check_pairs([96, 160, 112, 160])[0] is False
    assert B.check_pairs([96, 160, 112])[0] is False


def test_workspace_size_and_status_strings():
    layer = B.ModseLayer(2048, [2816, 8448, 3520, 7744, 4224, 7040, 4928, 6336], 2)
    a = layer.workspace_bytes(B.MODSE_BF16, 8192, False)
    b = layer.workspace_bytes(B.MODSE_BF16, 8192, True)
    c = layer.workspace_bytes(B.MODSE_BF16, 16384, True)
    assert 0 < a < b < c
    assert a % 256 == 0
    assert layer.workspace_bytes(B.MODSE_BF16, -1, True) == 0
    assert layer.workspace_bytes(7, 16, True) == 0
    layer.destroy()
    assert B.status_string(B.MODSE_OK) == "ok"
    assert "workspace" in B.status_string(B.MODSE_ERR_WORKSPACE_TOO_SMALL)


def test_forward_argument_errors_need_no_gpu():
    lib = B.load()
    layer = B.ModseLayer(64, [96, 160, 112, 144], 2)
    w = B._Weights(0x1000, 0x1000, 0x1000, 0x1000)
    n = layer.workspace_bytes(B.MODSE_F32, 16, True)
    f = lambda *a: lib.modse_forward(layer._h, *a)
    assert f(B.MODSE_F32, ctypes.byref(w), 0x1000, 0, 0x1000, 0x1000, n, 1, None) == B.MODSE_OK      # T = 0
    assert f(B.MODSE_F32, ctypes.byref(w), 0x1000, 16, 0x1000, 0x1000, n - 1, 1, None) == B.MODSE_ERR_WORKSPACE_TOO_SMALL
    assert f(B.MODSE_F32, ctypes.byref(w), 0x1000, 16, 0x1000, 0x1010, n, 1, None) == B.MODSE_ERR_INVALID_ARG   # ws align
    assert f(B.MODSE_F32, ctypes.byref(w), 0x1004, 16, 0x1000, 0x1000, n, 1, None) == B.MODSE_ERR_INVALID_ARG   # x align
    assert f(B.MODSE_F32, None, 0x1000, 16, 0x1000, 0x1000, n, 1, None) == B.MODSE_ERR_INVALID_ARG
    assert f(5, ctypes.byref(w), 0x1000, 16, 0x1000, 0x1000, n, 1, None) == B.MODSE_ERR_INVALID_ARG
    # bf16 needs widths that are multiples of 64 and a model width that is a multiple of 128
    assert f(B.MODSE_BF16, ctypes.byref(w), 0x1000, 16, 0x1000, 0x1000, n, 1, None) == B.MODSE_ERR_UNSUPPORTED
    g = B._WGrads(0x1000, 0x1000, 0x1000, 0x1000)
    st = lib.modse_backward(layer._h, B.MODSE_F32, ctypes.byref(w), 0x1000, 0x1000, 16, 0x1000, ctypes.byref(g),
                            0x1000, n, None)
    assert st == B.MODSE_ERR_STATE                                 # no forward was saved
    layer.destroy()


def test_noise_gate_argument_errors_need_no_gpu():
    lib = B.load()
    layer = B.ModseLayer(64, [96, 160, 112, 144], 2)
    cf = ctypes.c_float
    assert lib.modse_set_noise_gate(None, 0x1000, cf(1.0), cf(1e-6)) == B.MODSE_ERR_INVALID_ARG
    assert lib.modse_set_noise_gate(layer._h, 0x1004, cf(1.0), cf(1e-6)) == B.MODSE_ERR_INVALID_ARG   # alignment
    assert lib.modse_set_noise_gate(layer._h, 0x1000, cf(1.0), cf(-1.0)) == B.MODSE_ERR_INVALID_ARG   # eps < 0
    assert lib.modse_set_noise_gate(layer._h, 0x1000, cf(float("nan")), cf(0.0)) == B.MODSE_ERR_INVALID_ARG
    assert lib.modse_set_noise_gate(layer._h, 0x1000, cf(1.0), cf(1e-6)) == B.MODSE_OK
    assert lib.modse_set_noise_gate(layer._h, None, cf(0.0), cf(0.0)) == B.MODSE_OK                   # off again
    assert lib.modse_set_noise_grads(None, 0x1000, 0x1000) == B.MODSE_ERR_INVALID_ARG
    assert lib.modse_set_noise_grads(layer._h, 0x1000, 0x1000) == B.MODSE_OK
    layer.destroy()


def test_tile_plan_validation_needs_no_gpu():
    layer = B.ModseLayer(2048, [2816, 8448], 2)
    assert layer.tile_plan() == -1                      # library default until tuned or set
    layer.set_tile_plan(B.DEFAULT_TILE_PLAN)
    assert layer.tile_plan() == B.DEFAULT_TILE_PLAN
    layer.set_tile_plan(-1)
    assert layer.tile_plan() == -1
    layer.set_tile_plan(0x3F3F)
    assert layer.tile_plan() == 0x3F3F
    for bad in (-2, 0x4000, 0x40, 0x80):
        with pytest.raises(B.ModseError) as ei:
            layer.set_tile_plan(bad)
        assert ei.value.status == B.MODSE_ERR_INVALID_ARG
    layer.destroy()


def test_fusion_flags_and_debug_switches_need_no_gpu():
    layer = B.ModseLayer(2048, [2816, 8448], 2)
    assert layer.fusion() == 0
    layer.set_fusion(B.MODSE_FUSE_GATHER | B.MODSE_FUSE_DG_ROWDOT | B.MODSE_FUSE_SCATTER)
    assert layer.fusion() == 7
    with pytest.raises(B.ModseError) as ei:
        layer.set_fusion(8)
    assert ei.value.status == B.MODSE_ERR_INVALID_ARG
    layer.set_debug_checks(True)
    prow, guard, pmax = layer.debug_workspace_offsets(B.MODSE_BF16, 1000, True)
    assert prow % 256 == 0 and guard % 256 == 0 and pmax % 128 == 0 and pmax >= 2000
    # the guard blocks are part of the workspace in either mode
    n = layer.workspace_bytes(B.MODSE_BF16, 1000, True)
    layer.set_debug_checks(False)
    assert layer.workspace_bytes(B.MODSE_BF16, 1000, True) == n
    layer.destroy()
    B.debug_set_wait_limit_ms(2000)
    B.debug_skip_tile_loads(-1, -1)
    B.debug_set_dynamic_tiles(True)
    B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)
