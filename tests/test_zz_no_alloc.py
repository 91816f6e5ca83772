"""modse_route_static_scratch: routing for callers that may not allocate device memory
(plugins inside a framework callback, code inside a pool it does not own).  Its scratch is a
fixed array in the library, so this checks - through the C ABI, twice in a row on different
batches - that it returns exactly what the workspace-based modse_forward returns and what the
fp64 oracle's router returns, and that a batch too large for the array is refused instead of
overrunning it.

Collected last on purpose: a failure here leaves every other test already run."""
import ctypes

import numpy as np
import pytest

from oracle import modse_oracle as O
from paper_2409_12210_b200 import inputs as I

import helpers as H

pytestmark = pytest.mark.gpu


def routing_via_forward(inp):
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = inp.cfg
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    wr, wg, wu, wd = B.pack_weights(inp, "cuda")
    x = torch.from_numpy(inp.x).to("cuda", dt)
    y = torch.empty_like(x)
    ws = layer.alloc_workspace(dt, x.shape[0], False)
    layer.forward(wr, wg, wu, wd, x, y, ws, False)
    rt = {k: v.cpu().numpy().copy() for k, v in layer.get_routing(ws, x.shape[0]).items()}
    torch.cuda.synchronize()
    layer.destroy()
    return rt, x, wr


@pytest.mark.parametrize("name", ["tiny_f32", "bf16"])
def test_two_calls_in_a_row_match_the_workspace_path(name):
    import torch
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    if name == "tiny_f32":
        cfgs = [I.CONFIGS["tiny_f32"], I.with_tokens(I.CONFIGS["tiny_f32"], 77)]
    else:
        base = I.LayerConfig("na_bf16", "bf16", 256, (128, 384, 192, 320), 2, 1000, seed=5, weight_std=0.05)
        cfgs = [base, I.LayerConfig("na_bf16_b", "bf16", 256, (128, 384, 192, 320), 2, 333, seed=6, weight_std=0.05)]
    for cfg in cfgs:                                   # second call reuses the array the first one left dirty
        inp, _ = H.screened(cfg)                        # near-tie tokens re-drawn, as in every parity test
        ref, x, wr = routing_via_forward(inp)
        got = B.route_static_scratch(x, wr, cfg.top_k)
        torch.cuda.synchronize()
        for key in ("topk_idx", "counts", "counts_slot", "offsets", "row_of", "token_of"):
            np.testing.assert_array_equal(got[key].cpu().numpy(), ref[key], err_msg=f"{cfg.name}:{key}")
        np.testing.assert_array_equal(got["topk_gate"].cpu().numpy(), ref["topk_gate"])   # same kernels: same bits
        assert B.route_static_scratch_status() == B.MODSE_OK
        # and against the oracle's router (Eq. 2-3): tables bit-exact, gates within the derived bound
        rt = O.route(np.asarray(inp.x, np.float64), np.asarray(inp.w_router, np.float64), cfg.top_k)
        H.check_routing({k: v.cpu().numpy() for k, v in got.items()}, rt, inp)


def test_batches_beyond_the_fixed_array_are_refused():
    import torch
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    lib = B.load()
    cap = lib.modse_route_static_scratch_capacity()
    assert cap == 4 << 20
    x = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
    w = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    out = torch.zeros(16, dtype=torch.int32, device="cuda")
    p = out.data_ptr()
    st = lib.modse_route_static_scratch(B.MODSE_F32, 64, 4, 2, x.data_ptr(), w.data_ptr(), 5_000_000, p, p, p, p, p, p,
                                        p, None)
    assert st == B.MODSE_ERR_WORKSPACE_TOO_SMALL       # nothing was launched, nothing written
    st = lib.modse_route_static_scratch(B.MODSE_F32, 64, 4, 3, x.data_ptr(), w.data_ptr(), 64, p, p, p, p, p, p, p, None)
    assert st == B.MODSE_ERR_UNSUPPORTED
    torch.cuda.synchronize()
