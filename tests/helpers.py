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


def run_gpu(inp: I.LayerInputs, backward: bool, save: bool | None = None, out_f32: bool = False):
    """Forward (and backward) through the C ABI; returns host numpy results."""
    import torch
    from paper_2409_12210_b200 import binding as B
    cfg = inp.cfg
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    dev = "cuda"
    if "MODSE_TEST_PAIR_MASK" in os.environ:           # run the suite against the two-SM kernels
        B.debug_set_pair_kernels(int(os.environ["MODSE_TEST_PAIR_MASK"]))
    layer = B.ModseLayer(cfg.d_model, cfg.ffn_sizes, cfg.top_k)
    layer.set_output_f32(out_f32)
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


def check_routing(gpu_rt, rt, gate_tol=5e-6):
    for name in ("topk_idx", "counts", "counts_slot", "offsets", "row_of", "token_of"):
        np.testing.assert_array_equal(gpu_rt[name], getattr(rt, name), err_msg=name)
    assert np.max(np.abs(gpu_rt["topk_gate"] - rt.topk_gate)) <= gate_tol


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
    check_routing(gpu["routing"], ora["rt"])
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
