"""The failure paths of the library, each taken once in a form that cannot hang a GPU: a bounded wait that
runs out (nothing is in flight when it does), an index outside its table (checked, recorded, access skipped),
and an overwritten guard block between workspace regions (debug checks)."""
import numpy as np
import pytest

from paper_2409_12210_b200 import inputs as I

import helpers as H

pytestmark = pytest.mark.gpu

TINY_BF16 = I.LayerConfig("fail_tiny", "bf16", 128, (64, 128, 64, 128), 2, 200, seed=11, weight_std=0.05)


@pytest.fixture(scope="module", autouse=True)
def lib():
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    yield
    B.debug_set_wait_limit_ms(2000)
    B.debug_skip_tile_loads(-1, -1)
    B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)


def setup_layer(inp, save, slack_bytes=0):
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = inp.cfg
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    w = B.pack_weights(inp, "cuda")
    x = torch.from_numpy(inp.x).to("cuda", torch.bfloat16)
    y = torch.empty_like(x)
    n = layer.workspace_bytes(B.MODSE_BF16, x.shape[0], save)
    ws = torch.zeros(n + slack_bytes, dtype=torch.uint8, device="cuda")
    return layer, w, x, y, ws


@pytest.mark.parametrize("plan", [0x3F3A, 0b111010], ids=["cta_pairs", "one_cta"])
@pytest.mark.parametrize("product", [0, 1])
def test_a_wait_that_runs_out_is_reported_and_the_gpu_stays_usable(product, plan):
    """The producer of one CTA (of both CTAs of a pair) is told to load nothing for its first tile: no copy and no
    MMA of that CTA is in flight, its MMA warp waits for data that never comes, gives up after the (shortened)
    limit, the CTA frees its tensor memory and the kernel returns.  The host reads the time-out, and the next
    forward is correct."""
    import torch
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(TINY_BF16)
    layer, w, x, y, ws = setup_layer(inp, save=False)
    B.debug_set_default_tile_plan(plan)
    B.debug_set_wait_limit_ms(50)
    B.debug_skip_tile_loads(product, 0)
    try:
        layer.forward(*w, x, y, ws, False)                 # returns: the call only enqueues
        assert layer.check_device_status(ws) == B.MODSE_ERR_DEVICE_TIMEOUT
    finally:
        B.debug_set_wait_limit_ms(2000)
        B.debug_skip_tile_loads(-1, -1)
    layer.forward(*w, x, y, ws, False)
    assert layer.check_device_status(ws) == B.MODSE_OK
    torch.cuda.synchronize()
    ora = H.run_oracle(inp, backward=False)
    assert H.rel_err_beyond_storage(y.float().cpu().numpy(), ora["y"]) <= 2e-2
    layer.destroy()
    B.debug_set_default_tile_plan(B.DEFAULT_TILE_PLAN)


@pytest.mark.parametrize("fuse", [0, 2])
def test_a_row_index_outside_the_padded_rows_is_recorded_and_skipped(fuse):
    """One entry of the padded row table is overwritten from the host between forward and backward.  The
    workspace is allocated larger than needed, so that the planted row would still land in memory this test
    owns if a check were missing."""
    import torch
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(TINY_BF16)
    cfg = inp.cfg
    layer, w, x, y, ws = setup_layer(inp, save=True, slack_bytes=8 << 20)
    layer.set_fusion(fuse)
    layer.forward(*w, x, y, ws, True)
    assert layer.check_device_status(ws) == B.MODSE_OK
    prow_off, _, pmax = layer.debug_workspace_offsets(B.MODSE_BF16, cfg.n_tokens, True)
    table = ws[prow_off:prow_off + 4 * cfg.top_k * cfg.n_tokens].view(torch.int32)
    table[7] = pmax + 5                                     # 5 rows past the end: 5 * 128 * 4 bytes, inside the slack
    dy = torch.from_numpy(inp.dy).to("cuda", torch.bfloat16)
    dx = torch.empty_like(x)
    dwr = torch.empty(w[0].shape, dtype=torch.float32, device="cuda")
    dwg, dwu, dwd = (torch.empty_like(t) for t in w[1:])
    layer.backward(*w, x, dy, dx, dwr, dwg, dwu, dwd, ws)
    assert layer.check_device_status(ws) == B.MODSE_ERR_DEVICE_BOUNDS
    # the next forward clears the status word
    layer.forward(*w, x, y, ws, True)
    assert layer.check_device_status(ws) == B.MODSE_OK
    layer.destroy()


def test_an_overwritten_guard_block_is_reported_by_the_debug_checks():
    import torch
    from paper_2409_12210_b200 import binding as B
    inp, _ = H.screened(TINY_BF16)
    cfg = inp.cfg
    layer, w, x, y, ws = setup_layer(inp, save=True)
    layer.set_debug_checks(True)
    layer.forward(*w, x, y, ws, True)
    assert layer.check_device_status(ws) == B.MODSE_OK      # every guard block intact after a real forward
    _, guard_off, _ = layer.debug_workspace_offsets(B.MODSE_BF16, cfg.n_tokens, True)
    ws[guard_off:guard_off + 8] = 0                          # what a kernel writing past topk_idx would do
    assert layer.check_device_status(ws) == B.MODSE_ERR_DEVICE_BOUNDS
    layer.forward(*w, x, y, ws, True)                        # rewrites the guard blocks
    assert layer.check_device_status(ws) == B.MODSE_OK
    layer.destroy()
