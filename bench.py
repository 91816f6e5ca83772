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
NOMINAL_BF16_DENSE_TFLOPS = 2250.0     # vendor figure for dense bf16, the "bf16 dense peak" of the target
NOMINAL_HBM_GBS = 8000.0               # "~8 TB/s"
BURST_REGION_S = 1.0                   # timed regions shorter than this run on burst clocks: burst peak applies
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised in
# profiles/tc_grouped_gemm_pair_train_16k_ncu.md (one kernel and one launch per ncu run, --clock-control none);
# valid only for that workload, for the library's default tile plan and for the kernel source they were taken
# from (first 16 hex digits of the SHA-256 of csrc/tc_gemm.cu), otherwise "traffic" is reported as null.
NCU_TRAFFIC = {
    "workload": "train_16k", "tc_gemm_sha256_16": "4025bd8c15f9c71a",
    "bytes_per_launch": {"upgate_gemm_swiglu": 1.592e9, "down_gemm": 1.022e9, "down_dgrad_swiglu_bwd": 1.849e9,
                         "down_wgrad": 0.688e9, "upgate_dgrad": 1.976e9, "upgate_wgrad": 1.244e9},
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
    k, default = kinds[stage], B_DEFAULT_TILE_PLAN
    shape = lambda plan: 2 if (plan >> (8 + k)) & 1 else (plan >> k) & 1
    return shape(tile_plan) == shape(default)


B_DEFAULT_TILE_PLAN = 0x3F3A       # the library's default plan (binding.DEFAULT_TILE_PLAN)
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
    ap.add_argument("--tune", action="store_true",
                    help="set-up: let modse_tune_forward time the kernel shapes of the forward products on this GPU "
                         "(off by default: the library's default plan, CTA pairs everywhere, was the faster one inside "
                         "a forward + backward step on every board measured)")
    ap.add_argument("--no-tune", action="store_true", help="accepted and ignored: not tuning is the default")
    ap.add_argument("--no-equal-size", action="store_true",
                    help="skip the interleaved comparison with the equal-size layer of the same total width")
    ap.add_argument("--skew-pair", action="store_true",
                    help="also compare the skewed-routing stress workload with its equal-size twin")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the extra back-to-back run that gives the power-limited figure (0: skip)")
    ap.add_argument("--tile-plan", type=int, default=None,
                    help="tuning: bit k set = grouped product k on one-CTA 256-row tiles, bit 8 + k = on CTA-pair "
                         "tiles (skips the set-up tuning call)")
    ap.add_argument("--static-tiles", action="store_true",
                    help="tuning: deal tiles to the CTAs round-robin instead of handing them out from a counter")
    ap.add_argument("--epi16", type=int, nargs=3, default=None, metavar=("MASK128", "MASK256", "MASKPAIR"),
                    help="tuning: bit k set = grouped product k runs sixteen epilogue warps on 128-row / one-CTA "
                         "256-row / CTA-pair tiles")
    ap.add_argument("--fuse", type=int, default=0,
                    help="fusions across the permutation (sum of 1 gather, 2 dg row dot, 4 scatter-add; see modse.h)")
    ap.add_argument("--out-f32", action="store_true", help="write y, dx and the expert weight gradients as fp32")
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
    if args.tile_plan is not None:
        B.debug_set_default_tile_plan(args.tile_plan)
    if args.static_tiles:
        B.debug_set_dynamic_tiles(False)
    if args.epi16 is not None:
        B.debug_set_epilogue_warps(*args.epi16)
    dev = torch.device("cuda", local_rank)

    inp = I.generate(cfg)
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    T, d, K, W = cfg.n_tokens, cfg.d_model, args.steps, max(args.warmup, 3)
    L = max(1, args.layers)
    do_bwd = cfg.backward
    tune = dt == torch.bfloat16 and args.tune and args.tile_plan is None

    class Replica:
        """One layer with all its tensors resident on the device.  `host` holds seeded host tensors (the
        benchmark workload); without it only x and W_router are drawn on the host (they fix the routing) and
        the expert weights and dY are drawn on the device with the same distributions."""

        def __init__(self, c, host=None):
            self.cfg = c
            self.layer = B.ModseLayer(c.d_model, c.ffn_sizes, c.top_k)
            wstd = c.weight_std if c.weight_std is not None else c.d_model ** -0.5
            gen = torch.Generator(device=dev).manual_seed(c.seed + 977)
            rn = lambda shape, std: (torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std).to(dt)
            if host is not None:
                self.wr, self.wg, self.wu, self.wd = B.pack_weights(host, dev)
                self.x = torch.from_numpy(host.x).to(dev, dt)
                self.dy = torch.from_numpy(host.dy).to(dev, dt)
            else:
                ro = I.generate(c, routing_only=True)
                S = sum(c.ffn_sizes)
                self.x = torch.from_numpy(ro.x).to(dev, dt)
                self.wr = torch.from_numpy(ro.w_router).to(dev, dt)
                self.wg, self.wu, self.wd = rn((S, c.d_model), wstd), rn((S, c.d_model), wstd), rn((c.d_model, S), wstd)
                self.dy = rn(tuple(self.x.shape), 1.0)
            # layer-stack mode: layers 1.. get their own weights, tokens and upstream gradients (same
            # distributions, drawn on the device); no data flows between layers
            self.extra = []
            for l in range(1, L):
                self.extra.append((rn(tuple(self.wr.shape), wstd), rn(tuple(self.wg.shape), wstd),
                                   rn(tuple(self.wu.shape), wstd), rn(tuple(self.wd.shape), wstd),
                                   rn(tuple(self.x.shape), 1.0), rn(tuple(self.x.shape), 1.0)))
            odt = torch.float32 if args.out_f32 else dt
            self.y, self.dx = torch.empty(self.x.shape, dtype=odt, device=dev), torch.empty(self.x.shape, dtype=odt, device=dev)
            self.dwr = torch.empty(self.wr.shape, dtype=torch.float32, device=dev)
            self.dwg, self.dwu, self.dwd = (torch.empty(w.shape, dtype=odt, device=dev) for w in (self.wg, self.wu, self.wd))
            self.layer.set_output_f32(args.out_f32)
            self.layer.set_fusion(args.fuse)
            self.bwd = c.backward
            if args.noise_gate:
                w_noise = rn(tuple(self.wr.shape), c.d_model ** -0.5)
                self.noise = (w_noise, torch.empty(self.wr.shape, dtype=torch.float32, device=dev),
                              torch.empty(1, dtype=torch.float32, device=dev))
                self.layer.set_noise_gate(w_noise, 1.0, 1e-6)
                self.layer.set_noise_grads(self.noise[1], self.noise[2])
            if args.aux_alpha > 0:
                self.layer.set_aux_loss(args.aux_alpha)
            self.ws = self.layer.alloc_workspace(dt, c.n_tokens, self.bwd, dev)
            # set-up, outside every timed region: pick the tile shape of the forward products for this GPU
            if tune:
                self.layer.tune_forward(self.wr, self.wg, self.wu, self.wd, self.x, self.y, self.ws, self.bwd)
            self.tile_plan = self.layer.tile_plan()

        def step(self, xb=None, dyb=None, yb=None, dxb=None):
            ly = self.layer
            xb, dyb = (self.x if xb is None else xb), (self.dy if dyb is None else dyb)
            yb, dxb = (self.y if yb is None else yb), (self.dx if dxb is None else dxb)
            ly.forward(self.wr, self.wg, self.wu, self.wd, xb, yb, self.ws, self.bwd)
            n = ly.last_launch_count()
            if self.bwd:
                ly.backward(self.wr, self.wg, self.wu, self.wd, xb, dyb, dxb, self.dwr, self.dwg, self.dwu, self.dwd,
                            self.ws)
                n += ly.last_launch_count()
            for (wr_l, wg_l, wu_l, wd_l, x_l, dy_l) in self.extra:
                ly.forward(wr_l, wg_l, wu_l, wd_l, x_l, yb, self.ws, self.bwd)
                n += ly.last_launch_count()
                if self.bwd:
                    ly.backward(wr_l, wg_l, wu_l, wd_l, x_l, dy_l, dxb, self.dwr, self.dwg, self.dwu, self.dwd, self.ws)
                    n += ly.last_launch_count()
            return n

        def warm(self, n):
            for _ in range(n):
                launches = self.step()
            torch.cuda.synchronize()
            status = self.layer.check_device_status(self.ws)
            if status != 0:
                raise SystemExit(f"device status {status}: {B.status_string(status)}")
            self.counts = self.layer.get_routing(self.ws, self.cfg.n_tokens)["counts"].cpu().numpy()
            return launches

        def flops_step(self):
            fwd, bwd, _ = expert_flops(self.counts, self.cfg)
            return L * (fwd + (bwd if self.bwd else 0.0))      # layers 1.. route near-uniformly like layer 0

        def free(self):
            self.layer.destroy()

    main_rep = Replica(cfg, host=inp)
    layer, ws, x, tile_plan = main_rep.layer, main_rep.ws, main_rep.x, main_rep.tile_plan
    step = main_rep.step

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    launches_per_step = main_rep.warm(W)
    counts = main_rep.counts

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

    # ---- power-limited figure: the same steps back to back for a few seconds (clocks settle under the cap) ----
    sustained = None
    if args.sustained_seconds > 0:
        n_sus = max(K, int(args.sustained_seconds * 1e3 / ms_step) + 1)
        sampler_s = ClockSampler(local_rank)
        sync_all()
        sampler_s.start()
        ev0.record()
        for _ in range(n_sus):
            step()
        ev1.record()
        sync_all()
        clocks_s = sampler_s.stop()
        ms_sus = max_over_ranks(ev0.elapsed_time(ev1), dev) / n_sus
        sustained = {"steps": n_sus, "seconds": round(ms_sus * n_sus / 1e3, 3), "ms_per_step": ms_sus,
                     "value": whole_job_value(T, world, ms_sus), "unit": UNIT,
                     "tflops": main_rep.flops_step() / (ms_sus * 1e-3) / 1e12, "clocks": clocks_s}

    # ---- the equal-size layer of the same total width (and FLOPs), timed in this process, steps interleaved ----
    def ab_compare(rep_a, rep_b, n):
        """n rounds of (one step of a, one step of b), every step between its own pair of events."""
        rep_b.warm(W)
        rep_a.warm(1)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
        smp = ClockSampler(local_rank)
        sync_all()
        smp.start()
        for i in range(n):
            evs[i][0].record(); rep_a.step(); evs[i][1].record(); rep_b.step(); evs[i][2].record()
        sync_all()
        ck = smp.stop()
        ms_a = max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in evs) / n, dev)
        ms_b = max_over_ranks(sum(e[1].elapsed_time(e[2]) for e in evs) / n, dev)
        return ms_a, ms_b, ck

    def comparison(rep_a, cfg_b):
        rep_b = Replica(cfg_b)
        ms_a, ms_b, ck = ab_compare(rep_a, rep_b, K)
        fa, fb = rep_a.flops_step(), rep_b.flops_step()
        out = {"workload": rep_a.cfg.name, "equal_size_workload": cfg_b.name, "ffn_sizes_equal": list(cfg_b.ffn_sizes),
               "steps_each": K, "order": "interleaved, one step of each per round, own event pair per step",
               "ms_per_step": ms_a, "ms_per_step_equal": ms_b, "modse_over_equal": ms_a / ms_b,
               "tflops": fa / (ms_a * 1e-3) / 1e12, "tflops_equal": fb / (ms_b * 1e-3) / 1e12,
               "flops_ratio": fa / fb, "time_per_flop_ratio": (ms_a / fa) / (ms_b / fb),
               "counts": [int(c) for c in rep_a.counts], "counts_equal": [int(c) for c in rep_b.counts], "clocks": ck}
        rep_b.free()
        del rep_b
        torch.cuda.empty_cache()
        return out

    equal_size = skew_pair = None
    S_total = sum(cfg.ffn_sizes)
    if not args.no_equal_size and dt == torch.bfloat16 and S_total % (64 * cfg.n_experts) == 0 and \
            len(set(cfg.ffn_sizes)) > 1:
        from dataclasses import replace
        cfg_eq = replace(cfg, name=cfg.name + "_equal", ffn_sizes=(S_total // cfg.n_experts,) * cfg.n_experts)
        equal_size = comparison(main_rep, cfg_eq)
    if args.skew_pair and dt == torch.bfloat16:
        rep_sk = Replica(I.CONFIGS["train_16k_skew"] if args.tokens is None
                         else I.with_tokens(I.CONFIGS["train_16k_skew"], args.tokens))
        rep_sk.warm(W)
        cfg_b = I.CONFIGS["train_16k_equal_skew"]
        skew_pair = comparison(rep_sk, cfg_b if args.tokens is None else I.with_tokens(cfg_b, args.tokens))
        rep_sk.free()
        del rep_sk
        torch.cuda.empty_cache()

    # ---- end to end: pinned host inputs in, results out, every step ----
    dy = main_rep.dy
    hx, hdy = torch.from_numpy(inp.x).to(dt).pin_memory(), torch.from_numpy(inp.dy).to(dt).pin_memory()
    hy, hdx = torch.empty_like(main_rep.y, device="cpu").pin_memory(), torch.empty_like(main_rep.y, device="cpu").pin_memory()
    h2d = hx.numel() * hx.element_size() * (2 if do_bwd else 1)
    d2h = hy.numel() * hy.element_size() * (2 if do_bwd else 1)

    # Every step copies its inputs host -> device and its results device -> host; the copies of
    # neighbouring steps run on their own streams (two device buffers each way), as a data loader
    # that prefetches the next batch would.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    xin, dyin = [torch.empty_like(x) for _ in range(2)], [torch.empty_like(x) for _ in range(2)]
    yout, dxout = [torch.empty_like(main_rep.y) for _ in range(2)], [torch.empty_like(main_rep.y) for _ in range(2)]
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
    # no kernel of any timed region may have given up a wait or met a bad index: the numbers would mean nothing
    status = layer.check_device_status(ws)
    if status != 0:
        raise SystemExit(f"device status {status} after the timed regions: {B.status_string(status)}")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of every stage, and of the dominant one ----
    # Tensor stages are set against three denominators: the measured cuBLAS burst rate (a kernel timed alone
    # or in a short region, clocks near their maximum), the measured sustained rate (seconds under the power
    # cap) and the vendor's dense bf16 figure.  `frac` uses the measured one that fits the timed region.
    pk, pk_src = peaks()
    short_region = ms_total / 1e3 < BURST_REGION_S
    tensor_peak = pk["bf16_tflops"] if short_region else pk["bf16_tflops_sustained"]
    tensor_peak_kind = "burst" if short_region else "sustained"
    flops_step = main_rep.flops_step()
    work = stage_work(counts, cfg)
    stages = []
    for i in range(B.N_STAGES):
        vals = stage_ms[:, i]
        vals = vals[vals >= 0]
        if len(vals) == 0:
            continue
        ms = float(vals.mean())
        row = {"stage": B.stage_name(i), "ms": round(ms, 4), "bound": STAGE_BOUND[i]}
        if STAGE_BOUND[i] == "tensor":
            ach = work[i] / (ms * 1e-3) / 1e12
            row.update(achieved=round(ach, 1), unit="TFLOP/s", frac=round(ach / tensor_peak, 4),
                       frac_of_burst=round(ach / pk["bf16_tflops"], 4),
                       frac_of_sustained=round(ach / pk["bf16_tflops_sustained"], 4),
                       frac_of_dense_peak=round(ach / NOMINAL_BF16_DENSE_TFLOPS, 4))
        else:
            ach = work[i] / (ms * 1e-3) / 1e9
            row.update(achieved=round(ach, 1), unit="GB/s", frac=round(ach / pk["hbm_gbs"], 4),
                       frac_of_nominal=round(ach / NOMINAL_HBM_GBS, 4))
        stages.append(row)
    dom = max(stages, key=lambda s: s["ms"])
    roofline = {"kernel": dom["stage"], "bound": dom["bound"], "achieved": dom["achieved"],
                "peak": tensor_peak if dom["bound"] == "tensor" else pk["hbm_gbs"],
                "unit": dom["unit"], "frac": dom["frac"],
                "traffic": ncu_traffic(dom["stage"], cfg.name) if same_kernel_as_captured(dom["stage"], tile_plan) else None,
                "traffic_unit": "bytes per launch (ncu dram read + write)",
                "peak_source": (f"of {pk_src}, {tensor_peak_kind} cuBLAS bf16 rate (timed region {ms_total / 1e3:.2f} s)"
                                if dom["bound"] == "tensor" else f"of {pk_src} copy bandwidth"),
                "ms_per_launch": dom["ms"]}
    for key in ("frac_of_burst", "frac_of_sustained", "frac_of_dense_peak", "frac_of_nominal"):
        if key in dom:
            roofline[key] = dom[key]

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        tps, secs, cores = cpu_oracle_sample(inp, args.cpu_tokens)
        cpu = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": round(secs, 2),
               "sample": f"first {args.cpu_tokens} tokens of the workload as one batch, forward + full backward"}

    weight_mb = 3 * d * sum(cfg.ffn_sizes) * x.element_size() / 1e6
    act_mb = (3 if do_bwd else 1) * cfg.top_k * T * d * x.element_size() / 1e6
    tflops = flops_step / (ms_step * 1e-3) / 1e12
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "d_model": d, "ffn_sizes": list(cfg.ffn_sizes), "top_k": cfg.top_k,
                   "n_tokens": T, "layers": L, "noise_gate": bool(args.noise_gate), "aux_alpha": args.aux_alpha,
                   "tile_plan": tile_plan, "dynamic_tiles": not args.static_tiles, "epi16": args.epi16, "fuse": args.fuse,
                   "outputs": "fp32" if args.out_f32 else cfg.dtype,
                   "e2e_copies": "x, dY in and y, dx out of layer 0" if L > 1 else "x, dY in; y, dx out", "pass": "fwd+bwd" if do_bwd else "fwd", "parallelism": f"replicas x{world}",
                   "l2": f"inputs larger than L2: {weight_mb * L:.0f} MB of expert weights and {act_mb * L:.0f} MB of "
                         f"permuted activations are streamed per step (L2: 126 MB)"},
        "tflops": tflops,
        "tflops_frac_of_burst_peak": tflops / pk["bf16_tflops"],
        "tflops_frac_of_sustained_peak": tflops / pk["bf16_tflops_sustained"],
        "tflops_frac_of_dense_peak": tflops / NOMINAL_BF16_DENSE_TFLOPS,
        "peaks": {"source": pk_src, "bf16_tflops_burst": pk["bf16_tflops"],
                  "bf16_tflops_sustained": pk["bf16_tflops_sustained"], "hbm_gbs": pk["hbm_gbs"],
                  "bf16_tflops_dense_nominal": NOMINAL_BF16_DENSE_TFLOPS, "hbm_gbs_nominal": NOMINAL_HBM_GBS},
        "counts": [int(c) for c in counts],
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": ms_e2e / K},
        "gpu_launches": int(launches_per_step * K),
        "roofline": roofline,
        "stages": stages,
        "sustained": sustained,
        "equal_size": equal_size,
        "skew_pair": skew_pair,
        "cpu_baseline": cpu,
    }
    if sustained is not None:
        sustained["tflops_frac_of_sustained_peak"] = sustained["tflops"] / pk["bf16_tflops_sustained"]
        sustained["tflops_frac_of_dense_peak"] = sustained["tflops"] / NOMINAL_BF16_DENSE_TFLOPS
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
