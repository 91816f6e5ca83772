"""GPU parity of the second router term, H(x)_i = (x W_g)_i + RMSNorm(Softplus((x W_n)_i)) (Sec. 2, Eq. 2):
routing tables bit-exact, outputs and every gradient (dW_n and dgamma included) against the fp64 oracle."""
import dataclasses

import numpy as np
import pytest

from oracle import modse_oracle as O
from paper_2409_12210_b200 import inputs as I
from helpers import rel_err, rms_rel_err

pytestmark = pytest.mark.gpu

GAMMA, EPS = 0.75, 1e-6


def noisy_inputs(cfg: I.LayerConfig, tau=1e-4):
    """Seeded layer inputs plus W_n; tokens whose noisy logits are within tau of a routing tie are redrawn."""
    inp = I.generate(cfg)
    rng = np.random.default_rng(cfg.seed + 4242)
    wn = (rng.standard_normal((cfg.n_experts, cfg.d_model)) / np.sqrt(cfg.d_model)).astype(np.float32)
    if cfg.dtype == "bf16":
        wn = I.round_to_bf16(wn)
    f = lambda a: np.asarray(a, np.float64)
    x = f(inp.x)
    for _ in range(20):
        z = x @ f(inp.w_router).T + O.noise_term(x, f(wn), GAMMA, EPS)[0]
        bad = np.nonzero(O.routing_margin(z, cfg.top_k) <= tau)[0]
        if bad.size == 0:
            break
        x[bad] = f(inp.redraw_x(inp.rng, bad.size))
    else:
        raise AssertionError("could not clear near-ties")
    inp.x = x.astype(np.float32)
    return inp, wn


def oracle_noisy(inp, wn, backward=True):
    f = lambda a: np.asarray(a, np.float64)
    cfg = inp.cfg
    x, wr = f(inp.x), f(inp.w_router)
    wg = [f(w) for w in inp.w_gate]; wu = [f(w) for w in inp.w_up]; wd = [f(w) for w in inp.w_down]
    r, u = O.noise_term(x, f(wn), GAMMA, EPS)
    rt = O.route_from_logits(x @ wr.T + r, cfg.top_k)
    pw = O.pack_weights(wg, wu, wd)
    out = {"rt": rt, "y": O.forward_tokens(x, pw, rt)}
    if backward:
        g = O.backward(x, wr, wg, wu, wd, rt, f(inp.dy))
        dx_add, dwn, dgamma = O.noise_backward(x, f(wn), GAMMA, EPS, g.dz)
        # scale of dgamma's rounding error: dgamma is a signed sum of per-token terms dz.s / q
        sp = np.logaddexp(0.0, u)
        terms = (g.dz * sp).sum(1) / np.sqrt((sp ** 2).mean(1) + EPS)
        assert abs(terms.sum() - dgamma) <= 1e-9 * np.abs(terms).sum()
        out.update(g=g, dx=g.dx + dx_add, dw_noise=dwn, dgamma=dgamma, dgamma_scale=float(np.sqrt((terms ** 2).sum())))
    return out


def gpu_noisy(inp, wn, out_f32=False):
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = inp.cfg
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    odt = torch.float32 if (out_f32 or cfg.dtype == "f32") else dt
    dev = "cuda"
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    layer.set_output_f32(out_f32)
    wr, wg, wu, wd = B.pack_weights(inp, dev)
    wn_d = torch.from_numpy(wn).to(dev, dt)
    dwn = torch.full(wn.shape, float("nan"), dtype=torch.float32, device=dev)
    dgamma = torch.full((1,), float("nan"), dtype=torch.float32, device=dev)
    layer.set_noise_gate(wn_d, GAMMA, EPS)
    layer.set_noise_grads(dwn, dgamma)
    x = torch.from_numpy(inp.x).to(dev, dt)
    T = x.shape[0]
    y = torch.empty(x.shape, dtype=odt, device=dev)
    ws = layer.alloc_workspace(dt, T, True)
    layer.forward(wr, wg, wu, wd, x, y, ws, True)
    rt = {k: v.cpu().numpy().copy() for k, v in layer.get_routing(ws, T).items()}
    dy = torch.from_numpy(inp.dy).to(dev, dt)
    dx = torch.empty(x.shape, dtype=odt, device=dev)
    dwr = torch.empty(wr.shape, dtype=torch.float32, device=dev)
    dwg, dwu, dwd = (torch.empty(w.shape, dtype=odt, device=dev) for w in (wg, wu, wd))
    layer.backward(wr, wg, wu, wd, x, dy, dx, dwr, dwg, dwu, dwd, ws)
    torch.cuda.synchronize()
    out = dict(routing=rt, y=y.float().cpu().numpy(), dx=dx.float().cpu().numpy(), dw_router=dwr.cpu().numpy(),
               dw_noise=dwn.cpu().numpy(), dgamma=float(dgamma.item()), status=layer.check_device_status(ws))
    layer.destroy()
    return out


def check(gpu, ora, tol, tol_dx):
    for name in ("topk_idx", "counts", "counts_slot", "offsets", "row_of", "token_of"):
        np.testing.assert_array_equal(gpu["routing"][name], getattr(ora["rt"], name), err_msg=name)
    assert np.max(np.abs(gpu["routing"]["topk_gate"] - ora["rt"].topk_gate)) <= 5e-6
    assert gpu["status"] == 0
    errs = {"y": rel_err(gpu["y"], ora["y"]), "dx": rel_err(gpu["dx"], ora["dx"]),
            "dw_router": rel_err(gpu["dw_router"], ora["g"].dw_router),
            "dw_noise": rel_err(gpu["dw_noise"], ora["dw_noise"]),
            "dgamma": abs(gpu["dgamma"] - ora["dgamma"]) / ora["dgamma_scale"]}
    bad = {k: v for k, v in errs.items() if not (v <= (tol_dx if k in ("y", "dx") else tol))}
    assert not bad, (bad, errs)
    return errs


def test_noise_gate_changes_the_routing_of_the_test_inputs():
    """Guard against a vacuous test: with gamma = 0.75 a sizeable share of tokens picks other experts."""
    cfg = dataclasses.replace(I.CONFIGS["tiny_f32"])
    inp, wn = noisy_inputs(cfg)
    ora = oracle_noisy(inp, wn, backward=False)
    plain = O.route(np.asarray(inp.x, np.float64), np.asarray(inp.w_router, np.float64), cfg.top_k)
    assert (plain.topk_idx != ora["rt"].topk_idx).any(axis=1).mean() > 0.05


def test_noise_gate_f32_tiny():
    inp, wn = noisy_inputs(I.CONFIGS["tiny_f32"])
    check(gpu_noisy(inp, wn), oracle_noisy(inp, wn), 1e-4, 1e-4)


@pytest.mark.parametrize("n_experts", [8, 16])
def test_noise_gate_bf16(n_experts):
    """8 experts take the tensor-core router with W_n as a second n-tile; 16 experts take the FMA router."""
    base = I.CONFIGS["fwd_8k"]
    sizes = (256, 768, 384, 640, 512, 512, 320, 704) * (n_experts // 8)
    cfg = dataclasses.replace(base, name=f"noise_bf16_{n_experts}", backward=True, d_model=512, ffn_sizes=sizes, n_tokens=1500,
                              seed=91 + n_experts)
    inp, wn = noisy_inputs(cfg)
    gpu = gpu_noisy(inp, wn, out_f32=True)
    ora = oracle_noisy(inp, wn)
    check(gpu, ora, 2e-2, 2e-2)
    assert rms_rel_err(gpu["dw_noise"], ora["dw_noise"]) < 5e-3


def test_noise_gate_with_aux_loss_f32():
    """The auxiliary loss sees the same logits: its dense dz term flows into dW_n and dgamma too."""
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = I.CONFIGS["tiny_f32"]
    alpha = 2000.0
    inp, wn = noisy_inputs(cfg)
    f = lambda a: np.asarray(a, np.float64)
    x, wr = f(inp.x), f(inp.w_router)
    ora = oracle_noisy(inp, wn)
    _, _, _, dz_aux = O.aux_loss(ora["rt"].z, alpha)
    dz = ora["g"].dz + dz_aux
    dx_add, dwn, dgamma = O.noise_backward(x, f(wn), GAMMA, EPS, dz)
    dx_ref = ora["g"].dx + dz_aux @ wr + dx_add
    dev = "cuda"
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    layer.set_aux_loss(alpha)
    wrd, wg, wu, wd = B.pack_weights(inp, dev)
    wn_d = torch.from_numpy(wn).to(dev)
    dwn_d = torch.empty(wn.shape, dtype=torch.float32, device=dev)
    dgm = torch.empty(1, dtype=torch.float32, device=dev)
    layer.set_noise_gate(wn_d, GAMMA, EPS)
    layer.set_noise_grads(dwn_d, dgm)
    xd = torch.from_numpy(inp.x).to(dev)
    y = torch.empty_like(xd)
    ws = layer.alloc_workspace(torch.float32, xd.shape[0], True)
    layer.forward(wrd, wg, wu, wd, xd, y, ws, True)
    dx = torch.empty_like(xd); dwr = torch.empty_like(wrd)
    dwg, dwu, dwdn = (torch.empty_like(w) for w in (wg, wu, wd))
    layer.backward(wrd, wg, wu, wd, xd, torch.from_numpy(inp.dy).to(dev), dx, dwr, dwg, dwu, dwdn, ws)
    torch.cuda.synchronize()
    assert rel_err(dx.cpu().numpy(), dx_ref) <= 1e-4
    assert rel_err(dwn_d.cpu().numpy(), dwn) <= 1e-4
    assert abs(dgm.item() - dgamma) <= 1e-4 * max(abs(dgamma), ora["dgamma_scale"])
    assert rel_err(dwr.cpu().numpy(), ora["g"].dw_router + dz_aux.T @ x) <= 1e-4
    # the dense term is visible: without it dW_n would differ by far more than the tolerance
    assert rel_err(O.noise_backward(x, f(wn), GAMMA, EPS, ora["g"].dz)[1], dwn) > 1e-2
    layer.destroy()


def test_backward_state_checks():
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = I.CONFIGS["tiny_f32"]
    inp, wn = noisy_inputs(cfg)
    dev = "cuda"
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    wr, wg, wu, wd = B.pack_weights(inp, dev)
    x = torch.from_numpy(inp.x).to(dev)
    y = torch.empty_like(x)
    ws = layer.alloc_workspace(torch.float32, x.shape[0], True)
    wn_d = torch.from_numpy(wn).to(dev)
    layer.set_noise_gate(wn_d, GAMMA, EPS)
    layer.forward(wr, wg, wu, wd, x, y, ws, True)
    dx = torch.empty_like(x); dwr = torch.empty_like(wr)
    dwg, dwu, dwdn = (torch.empty_like(w) for w in (wg, wu, wd))
    dy = torch.from_numpy(inp.dy).to(dev)
    with pytest.raises(B.ModseError) as ei:                       # gradient buffers were never given
        layer.backward(wr, wg, wu, wd, x, dy, dx, dwr, dwg, dwu, dwdn, ws)
    assert ei.value.status == B.MODSE_ERR_INVALID_ARG
    layer.set_noise_gate(None)
    with pytest.raises(B.ModseError) as ei:                       # the forward ran with the term on
        layer.backward(wr, wg, wu, wd, x, dy, dx, dwr, dwg, dwu, dwdn, ws)
    assert ei.value.status == B.MODSE_ERR_STATE
    torch.cuda.synchronize()
    layer.destroy()
