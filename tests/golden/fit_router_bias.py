"""Writes tests/golden/router_bias_zipf.txt: per-expert router logit offsets that make the
assignment shares of the skewed-routing stress configuration follow rank^-1.2 (rank 1 = the
widest expert).  Calls only the fp64 oracle's router.  The offsets enter the layer without any
API change: the last input channel is the constant 1 and the last router column holds b_e.

    python tests/golden/fit_router_bias.py
"""
import os
import sys
from dataclasses import replace

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import modse_oracle as O                      # noqa: E402
from paper_2409_12210_b200 import inputs as I             # noqa: E402


def main():
    base = I.CONFIGS["train_16k"]
    widths = np.array(base.ffn_sizes)
    rank = np.empty(len(widths), int)
    rank[np.argsort(-widths)] = np.arange(1, len(widths) + 1)
    target = rank.astype(float) ** -1.2
    target /= target.sum()
    b = np.zeros(len(widths))
    share = None
    for it in range(40):
        b = I.round_to_bf16(b.astype(np.float32)).astype(np.float64)     # what the bf16 router weight will hold
        cfg = replace(base, router_bias=tuple(float(v) for v in b))
        inp = I.generate(cfg, routing_only=True)
        rt = O.route(inp.x.astype(np.float64), inp.w_router.astype(np.float64), cfg.top_k)
        share = rt.counts / rt.counts.sum()
        err = np.max(np.abs(share / target - 1.0))
        print(it, np.round(share, 4), f"max rel err {err:.4f}", flush=True)
        if err < 0.01:
            break
        b = b + 0.7 * np.log(target / np.maximum(share, 1e-6))
        b -= b.max()
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "router_bias_zipf.txt")
    with open(out, "w") as f:
        f.write("# written by tests/golden/fit_router_bias.py (oracle router only); one offset per expert of\n")
        f.write("# widths " + " ".join(str(w) for w in widths) + ", shares ~ rank^-1.2, rank 1 = widest\n")
        f.write("# target shares " + " ".join(f"{t:.4f}" for t in target) + "\n")
        f.write("# achieved      " + " ".join(f"{s:.4f}" for s in share) + "\n")
        f.write(" ".join(repr(float(v)) for v in b) + "\n")
    print("wrote", out)


if __name__ == "__main__":
    main()
