"""GPU parity at the full benchmark sizes (width 2048, 8 experts of diverse widths, top-2;
8192 tokens forward-only, 16384 and 65536 tokens forward+backward), in the launch configuration
bench.py times.  The routing tables are compared in full (bit-exact); floating outputs are
compared on tokens / weight-gradient rows that the fp64 oracle computes one by one, and
dW_router through the identity dW_router = dz^T x.

Where the samples sit: part of them is drawn uniformly, the rest is placed by construction on
the rows where the kernels' tiles change behaviour - the first and last row of every expert
group, the rows either side of 128- and 256-row tile seams, every row of each group's last
(ragged) 128-row block, the rows either side of the boundaries between the row groups that
the tile order forms for experts with more than 8192 rows, and for the weight gradients the
hidden units at the ends of every expert, around the 64/128/256-column seams and in the last
partial 128-column block."""
import os

import numpy as np
import pytest

from oracle import modse_oracle as O
from paper_2409_12210_b200 import inputs as I

import helpers as H

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
RAW_CAP_BF16 = 4e-2      # raw max|err|/RMS of tensors stored in bf16 (one store rounding of a 5-sigma element is 2e-2)
# uniformly drawn tokens per workload (the placed ones come on top)
N_RANDOM_TOKENS = {"train_16k": 512, "train_64k": 512}
N_RANDOM_TOKENS_DEFAULT = 128
N_RANDOM_ROWS_PER_EXPERT = 128


def f64(a):
    return np.asarray(a, dtype=np.float64)


def row_group_bounds(c, tile_rows, d):
    """Rows (inside an expert group of c rows) at which the tile order starts a new group of row
    tiles: groups hold at most 16 Mi elements of the row operand and are of equal size (+-1 tile)."""
    mt = (c + tile_rows - 1) // tile_rows
    per_group = max(1, ((16 << 20) // d) // tile_rows)
    n_g = (mt + per_group - 1) // per_group
    if n_g <= 1:
        return []
    base, extra = divmod(mt, n_g)
    sizes = [base + 1] * extra + [base] * (n_g - extra)
    return [int(b) * tile_rows for b in np.cumsum(sizes)[:-1]]


def edge_rows_of_group(c, d, rng):
    """Group-relative rows placed by construction, with a label each."""
    rows = {}
    if c == 0:
        return rows
    rows[0] = "first"
    rows[c - 1] = "last"
    seams = [s for s in range(128, c, 128)]
    pick = set(seams[:2] + seams[-2:])                                  # 128, 256 and the last two seams
    pick |= {s for s in seams if s % 256 == 0 and s >= c - 512}          # the last 256-row seams
    if len(seams) > 4:
        pick |= set(int(s) for s in rng.choice(seams, 4, replace=False))
    for s in sorted(pick):
        rows.setdefault(s - 1, f"seam{s}-")
        rows.setdefault(s, f"seam{s}+")
    for tile_rows in (128, 256):
        for b in row_group_bounds(c, tile_rows, d):
            if 0 < b < c:
                rows.setdefault(b - 1, f"rowgroup{b}-")
                rows.setdefault(b, f"rowgroup{b}+")
    for r in range(128 * ((c - 1) // 128), c):                           # the last, ragged 128-row block
        rows.setdefault(r, "ragged")
    return rows


def edge_hidden_units(h, rng):
    units = {0, h - 1}
    for s in (64, 128, 256):
        for m in (s - 1, s):
            if 0 <= m < h:
                units.add(m)
        last = (h - 1) // s * s                                          # last seam of this size
        for m in (last - 1, last):
            if 0 <= m < h:
                units.add(m)
    if h % 128:
        units |= set(range(h - h % 128, h))                              # the partial 128-column block
    units |= set(int(r) for r in rng.integers(0, h, N_RANDOM_ROWS_PER_EXPERT))
    return sorted(units)


def oracle_samples(inp, backward, seed=7):
    cfg = inp.cfg
    rng = np.random.default_rng(seed)
    x, wr = f64(inp.x), f64(inp.w_router)
    rt = O.route(x, wr, cfg.top_k)
    pw = O.pack_weights([f64(w) for w in inp.w_gate], [f64(w) for w in inp.w_up], [f64(w) for w in inp.w_down])
    n_rand = N_RANDOM_TOKENS.get(cfg.name, N_RANDOM_TOKENS_DEFAULT)
    placed, labels = set(), {}
    for e in range(cfg.n_experts):
        c, off = int(rt.counts[e]), int(rt.offsets[e])
        for r, lab in edge_rows_of_group(c, cfg.d_model, rng).items():
            t = int(rt.token_of[off + r])
            placed.add(t)
            labels[lab.rstrip("+-0123456789")] = labels.get(lab.rstrip("+-0123456789"), 0) + 1
    rand = set(int(t) for t in rng.choice(cfg.n_tokens, n_rand, replace=False))
    sel = np.array(sorted(placed | rand), np.int32)
    print(f"{cfg.name}: {len(sel)} tokens compared ({len(placed)} placed on tile edges {labels}, {n_rand} drawn)")
    out = {"rt": rt, "sel": sel, "n_placed": len(placed), "y": O.forward_tokens(x, pw, rt, sel)}
    if backward:
        dy = f64(inp.dy)
        out["dx"], out["dg"], dz = O.backward_tokens(x, wr, pw, rt, dy, sel)
        out["dz"] = np.take_along_axis(dz, rt.topk_idx[sel].astype(np.int64), 1)
        rows_e, rows_r = [], []
        for e, h in enumerate(cfg.ffn_sizes):
            u = edge_hidden_units(h, rng)
            rows_e += [e] * len(u)
            rows_r += u
        out["rows_e"], out["rows_r"] = np.array(rows_e, np.int32), np.array(rows_r, np.int32)
        print(f"{cfg.name}: {len(rows_r)} weight-gradient rows compared "
              f"({min(np.bincount(rows_e))}-{max(np.bincount(rows_e))} per expert)")
        out["dwg"], out["dwu"], out["dwd"] = O.wgrad_rows(x, pw, rt, dy, out["rows_e"], out["rows_r"])
    return out


def gather(gpu, ora, cfg, backward):
    """The GPU's values at the compared tokens / weight-gradient rows, keyed like the oracle's samples."""
    sel = ora["sel"]
    got = {"y": gpu["y"][sel]}
    if backward:
        hoff = np.concatenate([[0], np.cumsum(cfg.ffn_sizes)])
        rows = hoff[ora["rows_e"]] + ora["rows_r"]
        got.update(dx=gpu["dx"][sel], dg=gpu["dg"][sel], dz=gpu["dz"][sel], dwg=gpu["dw_gate"][rows],
                   dwu=gpu["dw_up"][rows], dwd=gpu["dw_down"][:, rows].T)
    return got


def error_table(got, ora, cfg, backward, err):
    errs = {"y": err(got["y"], ora["y"])}
    if backward:
        nd = cfg.d_model if cfg.router_bias is None else cfg.d_model - 1
        errs["dx"] = err(got["dx"][:, :nd], ora["dx"][:, :nd])
        if cfg.router_bias is not None:
            # The stress case feeds the logit offsets through a constant input channel whose router
            # weights are ~100x the others, so dx of that one channel is sum_j dz_j b_j: it carries
            # the relative error of dz (bf16-level, bounded above by its own entry) times |b|, and
            # is measured against its own RMS.
            errs["dx_bias_channel"] = err(got["dx"][:, nd:], ora["dx"][:, nd:])
        errs["dg"] = H.rel_err(got["dg"], ora["dg"])
        errs["dz"] = H.rel_err(got["dz"], ora["dz"])
        # each expert's weight gradient is a tensor of its own (their magnitudes differ with the token
        # counts): the compared rows are normalised expert by expert and the worst expert is reported
        per_expert = lambda g, ref: max(err(g[ora["rows_e"] == e], ref[ora["rows_e"] == e])
                                        for e in range(cfg.n_experts))
        errs["dw_gate"] = per_expert(got["dwg"], ora["dwg"])
        errs["dw_up"] = per_expert(got["dwu"], ora["dwu"])
        errs["dw_down"] = per_expert(got["dwd"], ora["dwd"])
    return errs


def store_floor(ora, cfg, backward):
    """The same error table for the oracle's own values rounded once to bf16: what the store alone costs."""
    r = lambda a: I.round_to_bf16(a.astype(np.float32)).astype(np.float64)
    stored = {k: (r(v) if k in ("y", "dx", "dwg", "dwu", "dwd") else v) for k, v in ora.items()
              if k in ("y", "dx", "dg", "dz", "dwg", "dwu", "dwd")}
    return error_table(stored, ora, cfg, backward, H.rel_err)


def compare(gpu, ora, cfg, backward, bf16_outputs):
    got = gather(gpu, ora, cfg, backward)
    raw = error_table(got, ora, cfg, backward, H.rel_err)
    kind = "bf16" if bf16_outputs else "fp32"
    print(f"{cfg.name} {kind} outputs, raw max|err|/RMS:", {k: round(v, 4) for k, v in raw.items()})
    if not bf16_outputs:
        bad = {k: v for k, v in raw.items() if not (v <= TOL_BF16)}
        assert not bad, f"over tolerance {TOL_BF16}: {bad} (all: {raw})"
        return raw
    # bf16 outputs.  (a) The error beyond the one rounding of the stored element keeps the bound.  (b) The raw
    # figure keeps the bound as stated wherever the store of the exact result leaves room for it (its own
    # floor - the oracle's values rounded once, same elements, same metric - is at most half the bound), and
    # (c) never exceeds a loose cap.
    beyond = error_table(got, ora, cfg, backward, H.rel_err_beyond_storage)
    floor = store_floor(ora, cfg, backward)
    print(f"{cfg.name} bf16 outputs, beyond one store rounding:", {k: round(v, 4) for k, v in beyond.items()})
    print(f"{cfg.name} store floor (oracle values rounded once to bf16):", {k: round(v, 4) for k, v in floor.items()})
    bad = {k: v for k, v in beyond.items() if not (v <= TOL_BF16)}
    assert not bad, f"over tolerance {TOL_BF16}: {bad} (all: {beyond})"
    bad = {k: (v, floor[k]) for k, v in raw.items() if floor[k] <= TOL_BF16 / 2 and not (v <= TOL_BF16)}
    assert not bad, f"raw error over {TOL_BF16} although the store floor is under half of it: {bad}"
    bad = {k: v for k, v in raw.items() if not (v <= RAW_CAP_BF16)}
    assert not bad, f"raw error over {RAW_CAP_BF16}: {bad}"
    return raw


@pytest.mark.parametrize("name", ["fwd_8k", "train_16k", "train_16k_skew", "table2_700m", "table2_300m", "train_64k"])
def test_full_size_sampled_parity(name):
    cfg = I.CONFIGS[name]
    inp, n_redrawn = H.screened(cfg)
    assert n_redrawn < 0.01 * cfg.n_tokens
    ora = oracle_samples(inp, cfg.backward)
    assert ora["n_placed"] * 4 >= len(ora["sel"])          # at least a quarter of the tokens sit on tile edges
    rt = ora["rt"]
    # near-uniform routing, as in the paper's summed-slot shares (every expert 0.118-0.133 of the assignments)
    share = rt.counts / rt.counts.sum()
    if cfg.router_bias is None:
        assert share.min() > 0.08 and share.max() < 0.17
    else:
        # stress case: shares ~ rank^-1.2 with the widest expert first (fitted offsets, 1 % of target)
        want = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "router_bias_zipf.txt"), comments=None,
                          skiprows=2, max_rows=1, usecols=range(3, 11))
        assert np.max(np.abs(share / want - 1.0)) < 0.02

    gpu32 = H.run_gpu(inp, cfg.backward, out_f32=True)
    assert gpu32["status"] == 0
    ge, gt = H.check_routing(gpu32["routing"], rt, inp)
    print(f"{cfg.name}: largest gate error {ge:.2e} (smallest per-token bound {gt:.2e})")
    compare(gpu32, ora, cfg, cfg.backward, bf16_outputs=False)

    gpu = H.run_gpu(inp, cfg.backward)
    assert gpu["status"] == 0
    H.check_routing(gpu["routing"], rt, inp)
    compare(gpu, ora, cfg, cfg.backward, bf16_outputs=True)

    if cfg.backward:
        # dW_router = dz^T x holds for any batch size; dz itself is checked on the sampled tokens above
        dz_full = np.zeros((cfg.n_tokens, cfg.n_experts))
        np.put_along_axis(dz_full, rt.topk_idx.astype(np.int64), f64(gpu["dz"]), 1)
        ref = dz_full.T @ f64(inp.x)
        assert H.rel_err(gpu["dw_router"], ref) < 1e-4
        # routing invariants at full size
        tok = gpu["routing"]["token_of"]
        assert np.array_equal(np.bincount(tok, minlength=cfg.n_tokens), np.full(cfg.n_tokens, cfg.top_k))
        assert np.allclose(gpu["routing"]["topk_gate"].sum(1), 1.0, atol=1e-6)


def test_unscreened_inputs_disagree_with_the_oracle_only_on_near_ties():
    """Without the re-drawing of near-tie tokens the fp32 router and the fp64 oracle may pick differently,
    but only where the oracle's own logit gap is below the screening margin."""
    import torch
    from paper_2409_12210_b200 import binding as B, build
    build.build()
    cfg = I.CONFIGS["train_16k"]
    inp = I.generate(cfg, routing_only=True)
    rt = O.route(f64(inp.x), f64(inp.w_router), cfg.top_k)
    x = torch.from_numpy(inp.x).to("cuda", torch.bfloat16)
    wr = torch.from_numpy(inp.w_router).to("cuda", torch.bfloat16)
    got = B.route_static_scratch(x, wr, cfg.top_k)
    torch.cuda.synchronize()
    idx = got["topk_idx"].cpu().numpy()
    differ = np.nonzero(np.any(idx != rt.topk_idx, axis=1))[0]
    margin = O.routing_margin(rt.z, cfg.top_k)
    print(f"unscreened train_16k: {len(differ)} tokens routed differently, largest oracle margin among them "
          f"{margin[differ].max() if len(differ) else 0.0:.2e}")
    assert np.all(margin[differ] < 1e-4)
    assert len(differ) < 0.01 * cfg.n_tokens
