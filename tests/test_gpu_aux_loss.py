"""Auxiliary load-balance loss (Sec. 3.2, Eq. 7-10) on the GPU against the fp64 oracle: the loss
value with f and P, and its gradient through the router (dx and dW_router) when it is switched
into the backward pass."""
import numpy as np
import pytest

from oracle import modse_oracle as O
from paper_2409_12210_b200 import inputs as I

import helpers as H

pytestmark = pytest.mark.gpu

ALPHA = 0.01       # Switch-Transformer scale; the paper does not print its alpha


def run(cfg, alpha, out_f32=True):
    import torch
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    inp, _ = H.screened(cfg)
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    odt = torch.float32 if out_f32 else dt
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    layer.set_output_f32(out_f32)
    layer.set_aux_loss(alpha)
    wr, wg, wu, wd = B.pack_weights(inp, "cuda")
    x = torch.from_numpy(inp.x).to("cuda", dt); dy = torch.from_numpy(inp.dy).to("cuda", dt)
    T = x.shape[0]
    y = torch.empty(x.shape, dtype=odt, device="cuda"); dx = torch.empty_like(y)
    dwr = torch.empty(wr.shape, dtype=torch.float32, device="cuda")
    dwg, dwu, dwd = (torch.empty(w.shape, dtype=odt, device="cuda") for w in (wg, wu, wd))
    ws = layer.alloc_workspace(dt, T, True)
    layer.forward(wr, wg, wu, wd, x, y, ws, True)
    loss, f, P = layer.aux_loss(ws, T, alpha)
    layer.backward(wr, wg, wu, wd, x, dy, dx, dwr, dwg, dwu, dwd, ws)
    torch.cuda.synchronize()
    assert layer.check_device_status(ws) == 0
    out = dict(loss=float(loss.item()), f=f.cpu().numpy(), P=P.cpu().numpy(), dx=dx.float().cpu().numpy(),
               dw_router=dwr.cpu().numpy())
    layer.destroy()
    return inp, out


@pytest.mark.parametrize("name,tol", [("tiny_f32", 1e-4), ("bf16", 2e-2)])
def test_aux_loss_value_and_router_gradient(name, tol):
    cfg = I.CONFIGS["tiny_f32"] if name == "tiny_f32" else \
        I.LayerConfig("aux_bf16", "bf16", 256, (128, 384, 192, 320), 2, 1000, seed=1, weight_std=0.05)
    # a large alpha makes the auxiliary part of the gradients comparable to the layer part
    alpha = 2000.0
    inp, gpu = run(cfg, alpha)
    ora = H.run_oracle(inp, True)
    x64, wr64 = inp.x.astype(np.float64), inp.w_router.astype(np.float64)
    loss, f, P, dz_aux = O.aux_loss(ora["rt"].z, alpha)
    assert abs(gpu["loss"] - loss) <= 1e-4 * abs(loss)
    np.testing.assert_allclose(gpu["f"], f, rtol=0, atol=1e-7)            # integer counts / T
    np.testing.assert_allclose(gpu["P"], P, rtol=1e-4, atol=1e-7)
    dx_ref = ora["g"].dx + dz_aux @ wr64
    dwr_ref = ora["g"].dw_router + dz_aux.T @ x64
    # the auxiliary part must be visible in the reference, else this would test nothing
    assert H.rel_err(dwr_ref, ora["g"].dw_router) > 0.05
    assert H.rel_err(gpu["dx"], dx_ref) <= tol
    assert H.rel_err(gpu["dw_router"], dwr_ref) <= tol


def test_alpha_zero_leaves_backward_unchanged():
    cfg = I.CONFIGS["tiny_f32"]
    _, a = run(cfg, 0.0)
    inp, _ = H.screened(cfg)
    b = H.run_gpu(inp, True)
    assert np.array_equal(a["dx"], b["dx"]) and np.array_equal(a["dw_router"], b["dw_router"])
    loss, f, P, _ = O.aux_loss(H.run_oracle(inp, False)["rt"].z, ALPHA)
    assert abs(a["f"].sum() - 1.0) < 1e-6 and abs(a["P"].sum() - 1.0) < 1e-5
