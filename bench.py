"""Benchmark of the MoDSE layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step is one pass of the whole layer - router, permutation, grouped up/gate
GEMM with SwiGLU, grouped down GEMM, combine, and the full backward - over one
batch of seeded synthetic tokens shaped like the paper's 700M x 8 model (width
2048, 8 experts, top-2).  Prints ONE JSON line.

N > 1 runs N independent replicas of the layer (one process per GPU under
torchrun): the layer runs on one GPU and has no exchange step, so throughput is
reported as weak scaling over replicas, timed as the maximum over ranks.

`--impl reference` times the fp64 CPU checker (the only other implementation
of this layer) on a bounded sample of the same workload, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2409_12210_b200 import inputs as I  # noqa: E402

METRIC = "modse_layer_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
# profiles/tc_grouped_gemm_train_16k_ncu_full.md; valid only for that workload and for the kernel source it was
# taken from (first 16 hex digits of the SHA-256 of csrc/tc_gemm.cu), otherwise "traffic" is reported as null.
NCU_TRAFFIC = {
    "workload": "train_16k", "tc_gemm_sha256_16": "c818e5c311c654cd",
    "bytes_per_launch": {"upgate_gemm_swiglu": 1.591e9, "down_gemm": 0.932e9, "down_dgrad_swiglu_bwd": 1.953e9,
                         "down_wgrad": 0.753e9, "upgate_dgrad": 1.910e9, "upgate_wgrad": 1.310e9},
}


def ncu_traffic(stage: str, workload: str):
    """DRAM bytes per launch from the committed ncu capture; None once the kernel source has changed since
    (the caller also drops it when a tile plan other than the captured default is in use)."""
    import hashlib
    try:
        src = os.path.join(ROOT, "paper_2409_12210_b200", "csrc", "tc_gemm.cu")
        digest = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    if workload != NCU_TRAFFIC["workload"] or digest != NCU_TRAFFIC["tc_gemm_sha256_16"]:
        return None
    return NCU_TRAFFIC["bytes_per_launch"].get(stage)


def same_kernel_as_captured(stage: str, tile_plan: int) -> bool:
    """True if `tile_plan` runs `stage` on the kernel variant of the ncu capture (the library's default plan)."""
    kinds = {"upgate_gemm_swiglu": 0, "down_gemm": 1, "down_dgrad_swiglu_bwd": 2, "down_wgrad": 3,
             "upgate_dgrad": 4, "upgate_wgrad": 5}
    if tile_plan < 0 or stage not in kinds:
        return True
    k, default = kinds[stage], 0x3A00
    return ((tile_plan >> k) & 1) == ((default >> k) & 1) and ((tile_plan >> (8 + k)) & 1) == ((default >> (8 + k)) & 1)


STAGE_BOUND = ["hbm", "hbm", "hbm", "tensor", "tensor", "hbm", "hbm", "tensor", "tensor", "tensor", "tensor", "hbm"]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def expert_flops(counts, cfg):
    """Algorithmic FLOPs of the expert GEMMs for the measured routing histogram:
    forward sum_e c_e * 6 d h_e, backward twice that; router 2TdN forward, 4TdN backward."""
    d, T, N = cfg.d_model, cfg.n_tokens, cfg.n_experts
    ch = float(sum(int(c) * h for c, h in zip(counts, cfg.ffn_sizes)))
    fwd = 6.0 * d * ch + 2.0 * T * d * N
    bwd = 12.0 * d * ch + 4.0 * T * d * N
    return fwd, bwd, ch


def stage_work(counts, cfg):
    """Algorithmic FLOPs (tensor-bound stages) or bytes (HBM-bound stages) per step, per stage."""
    d, T, N, k = cfg.d_model, cfg.n_tokens, cfg.n_experts, cfg.top_k
    ch = float(sum(int(c) * h for c, h in zip(counts, cfg.ffn_sizes)))
    R = k * T
    return [
        T * d * 2 + T * k * 12,                         # router: read x, write idx/gate/row tables
        T * k * 16,                                      # rank: integer tables
        T * d * 2 + R * d * 2,                           # permute: read x once, write k copies
        4.0 * d * ch,                                    # up/gate GEMM
        2.0 * d * ch,                                    # down GEMM
        R * d * 4 + T * d * 2,                           # combine: read fp32 rows, write y
        T * d * 2 + R * d * 4 + R * d * 2,               # dg + permute of dY
        2.0 * d * ch,                                    # down dgrad
        2.0 * d * ch,                                    # down wgrad
        4.0 * d * ch,                                    # up/gate dgrad
        4.0 * d * ch,                                    # up/gate wgrad
        T * d * 2 + R * d * 4 + T * d * 2,               # router backward: read x, dxp, write dx
    ]


class ClockSampler:
    """Reads SM clock, power and throttle reasons through NVML (read-only queries) every few
    milliseconds while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.stop_flag, self.thread, self.err = index, [], False, None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                      # no NVML: report that instead of clocks
            self.err = f"nvml unavailable: {type(e).__name__}"
            return
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    reasons = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                power = float(nv.nvmlDeviceGetPowerUsage(self.h)) / 1e3
                self.rows.append((sm, reasons, power))
            except Exception as e:
                self.err = f"nvml query failed: {type(e).__name__}"
                return
            time.sleep(0.004)

    def stop(self):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=1.0)
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": [self.err or "no samples"]}
        bits = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                0x2: "applications_clocks_setting", 0x10: "sync_boost", 0x80: "hw_power_brake_slowdown",
                0x100: "display_clock_setting"}                # 0x1 (gpu_idle) is not a limit and is left out
        seen = set()
        for _, r, _ in self.rows:
            for b, name in bits.items():
                if r & b:
                    seen.add(name)
            other = r & ~(sum(bits) | 0x1)
            if other:
                seen.add(f"other:0x{other:x}")
        return {"sm_mhz": float(np.median([r[0] for r in self.rows])), "sm_max_mhz": self.max_sm,
                "sm_mhz_range": [min(r[0] for r in self.rows), max(r[0] for r in self.rows)],
                "power_w_max": max(r[2] for r in self.rows), "samples": len(self.rows), "reasons": sorted(seen)}


def max_over_ranks(ms: float, device=None) -> float:
    """Largest per-rank time: the job's time is the slowest replica's (no-op for one process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas process world x tokens_per_rank tokens in the time of the slowest one."""
    return world * tokens_per_rank / (ms_per_step / 1e3)


def cpu_oracle_sample(inp, n_tok):
    """fp64 checker, forward + full backward, on the first n_tok tokens as one batch."""
    from oracle import modse_oracle as O
    f = lambda a: np.asarray(a, dtype=np.float64)
    x, dy = f(inp.x[:n_tok]), f(inp.dy[:n_tok])
    wr = f(inp.w_router)
    wg = [f(w) for w in inp.w_gate]; wu = [f(w) for w in inp.w_up]; wd = [f(w) for w in inp.w_down]
    t0 = time.perf_counter()
    y, rt = O.forward(x, wr, wg, wu, wd, inp.cfg.top_k)
    O.backward(x, wr, wg, wu, wd, rt, dy)
    dt = time.perf_counter() - t0
    return n_tok / dt, dt, O.num_threads()


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = I.generate(cfg)
    n_tok = args.ref_tokens
    for _ in range(args.warmup if args.warmup < 2 else 1):
        cpu_oracle_sample(inp, n_tok)
    times, cores = [], 1
    for _ in range(args.steps):
        tps, dt, cores = cpu_oracle_sample(inp, n_tok)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = n_tok / (ms / 1e3)
    sample = f"first {n_tok} tokens of the workload as one batch, forward + full backward"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "d_model": cfg.d_model, "ffn_sizes": list(cfg.ffn_sizes),
                   "top_k": cfg.top_k, "n_tokens": cfg.n_tokens, "pass": "fwd+bwd"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="train_16k", choices=sorted(I.CONFIGS))
    ap.add_argument("--cpu-tokens", type=int, default=256, help="tokens of the CPU baseline sample (about 15 s on 16 cores)")
    ap.add_argument("--ref-tokens", type=int, default=64,
                    help="--impl reference: tokens of the sample each step times (about 4 s on 16 cores)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tokens", type=int, default=None, help="override the workload's token count")
    ap.add_argument("--layers", type=int, default=1,
                    help="layer-stack sweep: a step runs this many independent layers (own weights, x and dY each)")
    ap.add_argument("--noise-gate", action="store_true",
                    help="add the second router term RMSNorm(Softplus(x W_n)) (Eq. 2) to the logits; off in the "
                         "default benchmark, whose router is x W_g alone")
    ap.add_argument("--aux-alpha", type=float, default=0.0,
                    help="coefficient of the auxiliary load-balance loss (Eq. 7) added to the objective in backward")
    ap.add_argument("--no-tune", action="store_true",
                    help="skip the set-up call that times the kernel shapes of the forward products on this GPU")
    ap.add_argument("--pair-mask", type=int, default=None,
                    help="tuning: which grouped products use the two-SM kernel (bit per product)")
    args = ap.parse_args()
    cfg = I.CONFIGS[args.workload]
    if args.tokens is not None:
        cfg = I.with_tokens(cfg, args.tokens)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2409_12210_b200 import binding as B, build as lib_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lib_build.build()
    if args.pair_mask is not None:
        B.debug_set_pair_kernels(args.pair_mask)
    dev = torch.device("cuda", local_rank)

    inp = I.generate(cfg)
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    T, d, K, W = cfg.n_tokens, cfg.d_model, args.steps, max(args.warmup, 3)
    layer = B.ModseLayer(d, cfg.ffn_sizes, cfg.top_k)
    wr, wg, wu, wd = B.pack_weights(inp, dev)
    x = torch.from_numpy(inp.x).to(dev, dt)
    dy = torch.from_numpy(inp.dy).to(dev, dt)
    # layer-stack mode: layers 1.. get their own seeded weights, tokens and upstream gradients, drawn on the
    # device with the same distributions (layer 0 is the workload's own tensors); no data flows between layers
    L = max(1, args.layers)
    extra = []
    for l in range(1, L):
        gen = torch.Generator(device=dev).manual_seed(cfg.seed + 1000 + l)
        rn = lambda ref, std: (torch.randn(ref.shape, generator=gen, device=dev, dtype=torch.float32) * std).to(dt)
        wstd = cfg.weight_std if cfg.weight_std is not None else d ** -0.5
        extra.append((rn(wr, wstd), rn(wg, wstd), rn(wu, wstd), rn(wd, wstd), rn(x, 1.0), rn(dy, 1.0)))
    y, dx = torch.empty_like(x), torch.empty_like(x)
    dwr = torch.empty(wr.shape, dtype=torch.float32, device=dev)
    dwg, dwu, dwd = torch.empty_like(wg), torch.empty_like(wu), torch.empty_like(wd)
    do_bwd = cfg.backward
    if args.noise_gate:
        gen = torch.Generator(device=dev).manual_seed(cfg.seed + 4242)
        w_noise = (torch.randn(wr.shape, generator=gen, device=dev, dtype=torch.float32) * d ** -0.5).to(dt)
        dw_noise = torch.empty(wr.shape, dtype=torch.float32, device=dev)
        dgamma = torch.empty(1, dtype=torch.float32, device=dev)
        layer.set_noise_gate(w_noise, 1.0, 1e-6)
        layer.set_noise_grads(dw_noise, dgamma)
    if args.aux_alpha > 0:
        layer.set_aux_loss(args.aux_alpha)
    ws = layer.alloc_workspace(dt, T, do_bwd, dev)
    # set-up, outside every timed region: pick the tile shape of the forward products for this GPU
    if dt == torch.bfloat16 and not args.no_tune and args.pair_mask is None:
        layer.tune_forward(wr, wg, wu, wd, x, y, ws, do_bwd)
    tile_plan = layer.tile_plan()

    def step(xb=None, dyb=None, yb=None, dxb=None):
        xb, dyb = (x if xb is None else xb), (dy if dyb is None else dyb)
        yb, dxb = (y if yb is None else yb), (dx if dxb is None else dxb)
        layer.forward(wr, wg, wu, wd, xb, yb, ws, do_bwd)
        n = layer.last_launch_count()
        if do_bwd:
            layer.backward(wr, wg, wu, wd, xb, dyb, dxb, dwr, dwg, dwu, dwd, ws)
            n += layer.last_launch_count()
        for (wr_l, wg_l, wu_l, wd_l, x_l, dy_l) in extra:
            layer.forward(wr_l, wg_l, wu_l, wd_l, x_l, yb, ws, do_bwd)
            n += layer.last_launch_count()
            if do_bwd:
                layer.backward(wr_l, wg_l, wu_l, wd_l, x_l, dy_l, dxb, dwr, dwg, dwu, dwd, ws)
                n += layer.last_launch_count()
        return n

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(W):
        launches_per_step = step()
    torch.cuda.synchronize()
    status = layer.check_device_status(ws)
    if status != 0:
        raise SystemExit(f"device status {status}: {B.status_string(status)}")
    counts = layer.get_routing(ws, T)["counts"].cpu().numpy()

    # ---- device-resident timing: K steps between two events, stages bracketed by the library's own events ----
    sampler = ClockSampler(local_rank)
    n_calls = K * L * (2 if do_bwd else 1)
    layer.stage_timing_begin(n_calls)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    sampler.start()
    ev0.record()
    for _ in range(K):
        step()
    ev1.record()
    sync_all()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    stage_ms = layer.stage_timing_end(n_calls)
    ms_total = max_over_ranks(ms_total, dev)
    ms_step = ms_total / K
    value = whole_job_value(T, world, ms_step)

    # ---- end to end: pinned host inputs in, results out, every step ----
    hx, hdy = torch.from_numpy(inp.x).to(dt).pin_memory(), torch.from_numpy(inp.dy).to(dt).pin_memory()
    hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
    h2d = hx.numel() * hx.element_size() * (2 if do_bwd else 1)
    d2h = hy.numel() * hy.element_size() * (2 if do_bwd else 1)

    # Every step copies its inputs host -> device and its results device -> host; the copies of
    # neighbouring steps run on their own streams (two device buffers each way), as a data loader
    # that prefetches the next batch would.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    xin, dyin = [torch.empty_like(x) for _ in range(2)], [torch.empty_like(x) for _ in range(2)]
    yout, dxout = [torch.empty_like(x) for _ in range(2)], [torch.empty_like(x) for _ in range(2)]
    E = lambda: [torch.cuda.Event() for _ in range(2)]
    ev_in, ev_done, ev_out = E(), E(), E()

    def load(b, first):
        with torch.cuda.stream(s_in):
            if not first:
                s_in.wait_event(ev_done[b])          # the step that last read this buffer pair is over
            xin[b].copy_(hx, non_blocking=True)
            if do_bwd:
                dyin[b].copy_(hdy, non_blocking=True)
            ev_in[b].record(s_in)

    def e2e_run(n_steps):
        comp = torch.cuda.current_stream()
        load(0, True)
        for i in range(n_steps):
            b = i & 1
            if i + 1 < n_steps:
                load((i + 1) & 1, i < 1)
            comp.wait_event(ev_in[b])
            if i >= 2:
                comp.wait_event(ev_out[b])           # results of step i-2 have left this buffer pair
            step(xin[b], dyin[b], yout[b], dxout[b])
            ev_done[b].record(comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[b])
                hy.copy_(yout[b], non_blocking=True)
                if do_bwd:
                    hdx.copy_(dxout[b], non_blocking=True)
                ev_out[b].record(s_out)
        comp.wait_stream(s_out)

    e2e_run(3)
    sync_all()
    ev0.record()
    e2e_run(K)
    ev1.record()
    sync_all()
    ms_e2e = ev0.elapsed_time(ev1)
    ms_e2e = max_over_ranks(ms_e2e, dev)
    e2e_value = whole_job_value(T, world, ms_e2e / K)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of every stage, and of the dominant one ----
    pk, pk_src = peaks()
    fwd_flops, bwd_flops, _ = expert_flops(counts, cfg)
    flops_step = L * (fwd_flops + (bwd_flops if do_bwd else 0.0))     # layers 1.. route near-uniformly like layer 0
    work = stage_work(counts, cfg)
    stages = []
    for i in range(B.N_STAGES):
        vals = stage_ms[:, i]
        vals = vals[vals >= 0]
        if len(vals) == 0:
            continue
        ms = float(vals.mean())
        if STAGE_BOUND[i] == "tensor":
            ach, peak, unit = work[i] / (ms * 1e-3) / 1e12, pk["bf16_tflops_sustained"], "TFLOP/s"
        else:
            ach, peak, unit = work[i] / (ms * 1e-3) / 1e9, pk["hbm_gbs"], "GB/s"
        stages.append({"stage": B.stage_name(i), "ms": round(ms, 4), "bound": STAGE_BOUND[i],
                       "achieved": round(ach, 1), "unit": unit, "frac": round(ach / peak, 4)})
    dom = max(stages, key=lambda s: s["ms"])
    roofline = {"kernel": dom["stage"], "bound": dom["bound"], "achieved": dom["achieved"],
                "peak": pk["bf16_tflops_sustained"] if dom["bound"] == "tensor" else pk["hbm_gbs"],
                "unit": dom["unit"], "frac": dom["frac"], "traffic": ncu_traffic(dom["stage"], cfg.name) if same_kernel_as_captured(dom["stage"], tile_plan) else None,
                "traffic_unit": "bytes per launch (ncu dram read + write)", "peak_source": f"of {pk_src}",
                "ms_per_launch": dom["ms"]}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        tps, secs, cores = cpu_oracle_sample(inp, args.cpu_tokens)
        cpu = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": round(secs, 2),
               "sample": f"first {args.cpu_tokens} tokens of the workload as one batch, forward + full backward"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "d_model": d, "ffn_sizes": list(cfg.ffn_sizes), "top_k": cfg.top_k,
                   "n_tokens": T, "layers": L, "noise_gate": bool(args.noise_gate), "aux_alpha": args.aux_alpha,
                   "tile_plan": tile_plan,
                   "e2e_copies": "x, dY in and y, dx out of layer 0" if L > 1 else "x, dY in; y, dx out", "pass": "fwd+bwd" if do_bwd else "fwd", "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (weights 554 MB, activations > 126 MB per step)"},
        "tflops": flops_step / (ms_step * 1e-3) / 1e12,
        "tflops_frac_of_sustained_peak": flops_step / (ms_step * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
        "counts": [int(c) for c in counts],
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": ms_e2e / K},
        "gpu_launches": int(launches_per_step * K),
        "roofline": roofline,
        "stages": stages,
        "cpu_baseline": cpu,
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
