"""The optional fusions across the permutation (modse_set_fusion), through the C ABI against the unfused
path and the fp64 oracle: the up/gate product gathering its rows from x, the gate gradient taken from the
down-dgrad epilogue, and the down / up-gate-dgrad products adding straight into y / dx."""
import numpy as np
import pytest

from paper_2409_12210_b200 import inputs as I

import helpers as H

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
ALL = ("y", "dx", "dw_router", "dw_gate", "dw_up", "dw_down", "dg", "dz")
# 1000 tokens: every expert group spans several 128-row tiles and ends in a ragged one; 2600: 256-row tiles with a
# second half present and absent
CASES = [I.LayerConfig("fuse_1000", "bf16", 256, (128, 384, 192, 320), 2, 1000, seed=1, weight_std=0.05),
         I.LayerConfig("fuse_2600", "bf16", 384, (448, 64, 320, 192), 2, 2600, seed=3, weight_std=0.05),
         I.LayerConfig("fuse_top1", "bf16", 256, (128, 384, 192), 1, 2100, seed=4, weight_std=0.05)]


@pytest.fixture(scope="module", autouse=True)
def lib():
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    yield
    B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("plan", [0, 63, 0x3F00])
def test_gathering_up_gate_product_gives_the_same_bits(cfg, plan):
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(cfg)
    B.debug_set_default_tile_plan(plan)
    try:
        ref = H.run_gpu(inp, True)
        got = H.run_gpu(inp, True, fuse=B.MODSE_FUSE_GATHER)
        ref_fwd = H.run_gpu(inp, False)
        got_fwd = H.run_gpu(inp, False, fuse=B.MODSE_FUSE_GATHER)     # no permute kernel at all
    finally:
        B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)
    for k in ALL:
        assert np.array_equal(ref[k], got[k]), k
    assert np.array_equal(ref_fwd["y"], got_fwd["y"]) and np.array_equal(ref["y"], got_fwd["y"])
    assert got_fwd["launches_fwd"] == ref_fwd["launches_fwd"] - 1
    assert got["status"] == 0 and got_fwd["status"] == 0
    H.check_all(inp, got, H.run_oracle(inp, True), TOL_BF16, discount_storage_rounding=True)


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("plan", [0, 63, 0x3F00])
def test_gate_gradient_from_the_down_dgrad_epilogue(cfg, plan):
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(cfg)
    B.debug_set_default_tile_plan(plan)
    try:
        ref = H.run_gpu(inp, True, out_f32=True)
        got = H.run_gpu(inp, True, out_f32=True, fuse=B.MODSE_FUSE_DG_ROWDOT)
    finally:
        B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)
    # everything that does not depend on dg is the same bits; dg itself is summed in another order
    for k in ("y", "dw_gate", "dw_up", "dw_down"):
        assert np.array_equal(ref[k], got[k]), k
    assert H.rel_err(got["dg"], ref["dg"]) < 1e-5
    ora = H.run_oracle(inp, True)
    H.check_all(inp, got, ora, TOL_BF16)
    assert got["launches_bwd"] == ref["launches_bwd"] + 1       # the kernel that sums the partial row dots


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("plan", [0, 63, 0x3F00])
def test_scatter_adding_epilogues_give_the_same_bits_as_the_combine_kernels(cfg, plan):
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(cfg)
    B.debug_set_default_tile_plan(plan)
    try:
        ref = H.run_gpu(inp, True, out_f32=True, fuse=B.MODSE_FUSE_DG_ROWDOT)
        got = H.run_gpu(inp, True, out_f32=True, fuse=B.MODSE_FUSE_SCATTER)
        again = H.run_gpu(inp, True, out_f32=True, fuse=B.MODSE_FUSE_SCATTER | B.MODSE_FUSE_GATHER)
        bf16_out = H.run_gpu(inp, True, fuse=B.MODSE_FUSE_SCATTER)    # flag does not apply to bf16 outputs: ignored
        plain = H.run_gpu(inp, True)
    finally:
        B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)
    for k in ALL:
        assert np.array_equal(ref[k], got[k]), k           # two addends into a zeroed element: order cannot matter
        assert np.array_equal(got[k], again[k]), k         # run to run, with the atomics
        assert np.array_equal(bf16_out[k], plain[k]), k
    assert got["launches_fwd"] == ref["launches_fwd"] - 1   # no combine kernel
    assert got["status"] == 0
    H.check_all(inp, got, H.run_oracle(inp, True), TOL_BF16)
