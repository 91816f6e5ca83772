"""Shared helpers of the GPU parity tests: run the CUDA library through its
Python binding and the fp64 oracle on the same seeded inputs."""
from __future__ import annotations

import os

import numpy as np

from oracle import modse_oracle as O
from paper_2409_12210_b200 import inputs as I


def screened(cfg: I.LayerConfig, tau: float = 1e-4):
    """Seeded inputs of `cfg` with near-tie tokens re-drawn (the fp64 oracle and an
    fp32-accumulating router may legitimately disagree below the margin)."""
    inp = I.generate(cfg)
    x, n = O.screen_inputs(inp.x.astype(np.float64), inp.w_router.astype(np.float64), cfg.top_k, inp.rng,
                           lambda r, m: inp.redraw_x(r, m).astype(np.float64), tau=tau)
    inp.x = x.astype(np.float32)
    return inp, n


def rel_err(got, ref) -> float:
    """max |got - ref| / RMS(ref)."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    if rms == 0.0:
        return float(np.max(np.abs(got - ref))) if ref.size else 0.0
    return float(np.max(np.abs(got - ref)) / rms)


def rel_err_beyond_storage(got, ref) -> float:
    """Like rel_err, but the part of each element's error that one bf16 rounding of the
    stored result explains (at most 2^-8 |ref|) is not counted.  For heavy-tailed tensors
    (weight gradients summed over a handful of tokens) that rounding alone exceeds any
    RMS-relative bound, whatever computed the value."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    if not ref.size:
        return 0.0
    rms = float(np.sqrt(np.mean(ref ** 2)))
    excess = np.maximum(0.0, np.abs(got - ref) - np.abs(ref) * 2.0 ** -8)
    return float(excess.max() / rms) if rms > 0 else float(excess.max())


def rms_rel_err(got, ref) -> float:
    """RMS(got - ref) / RMS(ref)."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0
    err = float(np.sqrt(np.mean((got - ref) ** 2))) if ref.size else 0.0
    return err / rms if rms > 0 else err


def run_gpu(inp: I.LayerInputs, backward: bool, save: bool | None = None, out_f32: bool = False, fuse: int = 0):
    """Forward (and backward) through the C ABI; returns host numpy results."""
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = inp.cfg
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    dev = "cuda"
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    layer.set_output_f32(out_f32)
    layer.set_fusion(fuse)
    odt = torch.float32 if out_f32 else dt
    wr, wg, wu, wd = B.pack_weights(inp, dev)
    x = torch.from_numpy(inp.x).to(dev, dt)
    T = x.shape[0]
    y = torch.empty(x.shape, dtype=odt, device=dev)
    save = backward if save is None else save
    ws = layer.alloc_workspace(dt, T, save)
    layer.forward(wr, wg, wu, wd, x, y, ws, save)
    out = {"launches_fwd": layer.last_launch_count()}
    rt = layer.get_routing(ws, T)
    torch.cuda.synchronize()
    out["y"] = y.float().cpu().numpy()
    out["routing"] = {k: v.cpu().numpy().copy() for k, v in rt.items()}
    if backward:
        dy = torch.from_numpy(inp.dy).to(dev, dt)
        dx = torch.empty(x.shape, dtype=odt, device=dev)
        dwr = torch.empty(wr.shape, dtype=torch.float32, device=dev)
        dwg, dwu, dwd = (torch.empty(w.shape, dtype=odt, device=dev) for w in (wg, wu, wd))
        layer.backward(wr, wg, wu, wd, x, dy, dx, dwr, dwg, dwu, dwd, ws)
        out["launches_bwd"] = layer.last_launch_count()
        dg, dz = layer.get_gate_grads(ws, T)
        torch.cuda.synchronize()
        out.update(dx=dx.float().cpu().numpy(), dw_router=dwr.cpu().numpy(), dw_gate=dwg.float().cpu().numpy(),
                   dw_up=dwu.float().cpu().numpy(), dw_down=dwd.float().cpu().numpy(), dg=dg.cpu().numpy().copy(),
                   dz=dz.cpu().numpy().copy())
    out["status"] = layer.check_device_status(ws)
    layer.destroy()
    return out


def run_oracle(inp: I.LayerInputs, backward: bool):
    f = lambda a: np.asarray(a, dtype=np.float64)
    wg = [f(w) for w in inp.w_gate]; wu = [f(w) for w in inp.w_up]; wd = [f(w) for w in inp.w_down]
    y, rt = O.forward(f(inp.x), f(inp.w_router), wg, wu, wd, inp.cfg.top_k)
    out = {"y": y, "rt": rt}
    if backward:
        out["g"] = O.backward(f(inp.x), f(inp.w_router), wg, wu, wd, rt, f(inp.dy))
    return out


def gate_tolerance(inp, rt):
    """Per-token bound on |gate_gpu - gate_oracle|, from the order in which the router adds its products.

    A gate is sigmoid(z_0 - z_1) (k = 2), whose slope is at most 1/4, so its error is at most a quarter of
    the two logits' errors plus the rounding of exp and of the division (a few units of 2^-24).  A logit
    is a sum of d products (exact in fp32 for bf16 operands, rounded once for fp32 ones) added in n_add
    fp32 steps; each step errs by at most one unit in the last place of the running sum (2^-23 of its
    magnitude; tensor-core accumulators may truncate, so no half-ulp is assumed).  The running sums are
    bounded here by P_j, the largest magnitude among the prefix sums of the products of logit j,
      - bf16, <= 16 experts, d % 128 == 0 (tensor-core router): four warps each add a quarter of the
        columns, 16 columns per step, then the quarters are added in order: n_add = d/64 + 3, P_j from the
        prefix sums in that order;
      - otherwise (fp32-FMA router): a lane adds every 32nd 8-column chunk with FMAs, then a 5-step butterfly:
        n_add = d/32 + 5, P_j bounded by sum_c |x_c w_jc| (valid for any order)."""
    cfg = inp.cfg
    x = np.asarray(inp.x, np.float64); w = np.asarray(inp.w_router, np.float64)
    T, d = x.shape
    k = cfg.top_k
    if k == 1:
        return np.zeros(T)
    idx = rt.topk_idx.astype(np.int64)
    P = np.zeros((T, k))
    tensor_core_router = cfg.dtype == "bf16" and cfg.n_experts <= 16 and d % 128 == 0
    for j in range(k):
        prod = x * w[idx[:, j]]                                     # [T, d]
        if tensor_core_router:
            # quarter q, 32-column block b, lane group tq (8 columns), half hf (4 columns): one step adds the 16
            # columns {b, all tq, one hf}
            steps = prod.reshape(T, 4, d // 128, 4, 2, 4).sum(axis=(3, 5)).reshape(T, 4, -1)   # [T, 4, d/64]
            pre = np.cumsum(steps, axis=2)
            quarters = np.cumsum(pre[:, :, -1], axis=1)
            P[:, j] = np.maximum(np.abs(pre).max(axis=(1, 2)), np.abs(quarters).max(axis=1))
            n_add = d // 64 + 3
        else:
            P[:, j] = np.abs(prod).sum(axis=1)
            n_add = d // 32 + 5 + (0 if cfg.dtype == "bf16" else 1)  # fp32 products are rounded too
    return 0.25 * n_add * 2.0 ** -23 * P.sum(axis=1) + 4 * 2.0 ** -24


def check_routing(gpu_rt, rt, inp=None):
    """Routing tables bit-exact; gates within the bound gate_tolerance derives (5e-6 where the inputs are
    not at hand, the size of that bound for 2048 columns and logits of magnitude 3)."""
    for name in ("topk_idx", "counts", "counts_slot", "offsets", "row_of", "token_of"):
        np.testing.assert_array_equal(gpu_rt[name], getattr(rt, name), err_msg=name)
    err = np.abs(gpu_rt["topk_gate"] - rt.topk_gate).max(axis=1)
    tol = gate_tolerance(inp, rt) if inp is not None else np.full(len(err), 5e-6)
    worst = int(np.argmax(err - tol)) if len(err) else 0
    assert np.all(err <= tol), f"gate error {err[worst]:.3e} over its bound {tol[worst]:.3e} at token {worst}"
    return float(err.max()) if len(err) else 0.0, float(tol.min()) if len(tol) else 0.0


def reference_tensors(ora):
    """Oracle results in the library's layouts, keyed like run_gpu's output."""
    ref = {"y": ora["y"]}
    if "g" in ora:
        g, rt = ora["g"], ora["rt"]
        ref.update(dx=g.dx, dw_router=g.dw_router, dw_gate=np.concatenate(g.dw_gate, 0),
                   dw_up=np.concatenate(g.dw_up, 0), dw_down=np.concatenate(g.dw_down, 1), dg=g.dg,
                   dz=np.take_along_axis(g.dz, rt.topk_idx.astype(np.int64), 1))
    return ref


def check_rms(gpu, ora, tol, skip=()):
    """RMS error of every tensor relative to the tensor's RMS (the typical, not the worst, element)."""
    errs = {k: rms_rel_err(gpu[k], v) for k, v in reference_tensors(ora).items() if k in gpu and k not in skip}
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, f"RMS error over {tol}: {bad} (all: {errs})"
    return errs


def check_all(inp, gpu, ora, tol, discount_storage_rounding=False, only=None):
    """Element-by-element comparison of every output (or of those named in `only`);
    returns the error table.  With discount_storage_rounding the tensors stored in
    bf16 are measured with rel_err_beyond_storage."""
    check_routing(gpu["routing"], ora["rt"], inp)
    full = rel_err
    rel_err_ = rel_err_beyond_storage if discount_storage_rounding else rel_err
    errs = {"y": rel_err_(gpu["y"], ora["y"])}
    if "dx" in gpu:
        g = ora["g"]
        rt = ora["rt"]
        errs["dx"] = rel_err_(gpu["dx"], g.dx)
        errs["dw_router"] = full(gpu["dw_router"], g.dw_router)
        errs["dw_gate"] = rel_err_(gpu["dw_gate"], np.concatenate(g.dw_gate, 0))
        errs["dw_up"] = rel_err_(gpu["dw_up"], np.concatenate(g.dw_up, 0))
        errs["dw_down"] = rel_err_(gpu["dw_down"], np.concatenate(g.dw_down, 1))
        errs["dg"] = full(gpu["dg"], g.dg)
        dz_kept = np.take_along_axis(g.dz, rt.topk_idx.astype(np.int64), 1)
        errs["dz"] = full(gpu["dz"], dz_kept)
    assert gpu["status"] == 0
    if only is not None:
        errs = {k: v for k, v in errs.items() if k in only}
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, f"over tolerance {tol}: {bad} (all: {errs})"
    return errs


def wgrad_errors_per_expert(inp, gpu, ora, err=rel_err):
    """max|err| / RMS(ref) of the three expert weight gradients, expert by expert (each expert's gradient is a
    tensor of its own: its magnitude follows the number of tokens routed to it).  Returns
    {tensor: [error of expert 0, ...]}; experts without tokens report the largest absolute entry (must be 0)."""
    g = ora["g"]
    hoff = np.concatenate([[0], np.cumsum(inp.cfg.ffn_sizes)])
    out = {"dw_gate": [], "dw_up": [], "dw_down": []}
    for e in range(inp.cfg.n_experts):
        a, b = int(hoff[e]), int(hoff[e + 1])
        out["dw_gate"].append(err(gpu["dw_gate"][a:b], g.dw_gate[e]))
        out["dw_up"].append(err(gpu["dw_up"][a:b], g.dw_up[e]))
        out["dw_down"].append(err(gpu["dw_down"][:, a:b], g.dw_down[e]))
    return out


def check_wgrads_per_expert(inp, gpu, ora, tol, min_tokens=256, few_tokens=32, err=rel_err):
    """Asserts the max bound on every expert's weight gradients separately (experts without any assignment
    must have exactly zero gradients).  A gradient summed over few tokens is heavy-tailed - its largest entries
    and its largest rows sit many RMS out, and the one bf16 rounding of their operands (dA, dB, Hm) alone passes
    an RMS-relative bound - so experts with `few_tokens` .. `min_tokens` - 1 assignments are held to twice the
    bound (a wrong tile tail is an error of order one, far beyond either), fewer to the pooled RMS bound only."""
    table = wgrad_errors_per_expert(inp, gpu, ora, err)
    counts = ora["rt"].counts
    bad = {}
    for name, errs in table.items():
        for e, v in enumerate(errs):
            if counts[e] == 0:
                assert v == 0.0, (name, e, v)
            elif counts[e] >= min_tokens and not (v <= tol):
                bad[(name, e, int(counts[e]))] = v
            elif counts[e] >= few_tokens and not (v <= 2 * tol):
                bad[(name, e, int(counts[e]))] = v
    assert not bad, f"per-expert weight-gradient error over {tol} (2x below {min_tokens} tokens): {bad}"
    return {name: max((v for e, v in enumerate(errs) if counts[e] >= few_tokens), default=0.0)
            for name, errs in table.items()}
