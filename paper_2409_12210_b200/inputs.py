"""Seeded synthetic inputs for the MoDSE layer.

This module only draws random tensors and rounds them to the storage type.  It
contains none of the layer's arithmetic, so both the CUDA library's callers and
the CPU checker can take their inputs from it.

Shapes follow the paper's 700M x 8 row of Table 1 (model width 2048, 8 experts,
top-2); expert widths are diverse with adjacent pairs of equal sum (Sec. 3.1,
Eq. 5-6).  Tensors are drawn from ``numpy.random.default_rng(seed)`` in the fixed
order x, W_router, W_gate[0..N), W_up[0..N), W_down[0..N), dY.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np


@dataclass(frozen=True)
class LayerConfig:
    name: str
    dtype: str                 # "f32" or "bf16": storage type of activations and expert weights
    d_model: int
    ffn_sizes: tuple
    top_k: int
    n_tokens: int
    seed: int = 0
    weight_std: float | None = None   # None: variance 1/fan_in; else this std for every weight
    router_bias: tuple | None = None  # per-expert logit offset carried by a constant input channel
    backward: bool = True

    @property
    def n_experts(self) -> int:
        return len(self.ffn_sizes)


WIDTHS_700M = (2816, 8448, 3520, 7744, 4224, 7040, 4928, 6336)   # pair sums 11264, ratio 3
WIDTHS_EQUAL = (5632,) * 8                                        # same total width, ratio 1
WIDTHS_RATIO2 = (3776, 7488, 4224, 7040, 4736, 6528, 5184, 6080)
WIDTHS_RATIO4 = (2240, 9024, 3072, 8192, 3968, 7296, 4800, 6464)
WIDTHS_TABLE2_700M = (9216, 1024, 8192, 2048, 6144, 4096, 5120, 5120)   # Table 2, 700M x 8
WIDTHS_TABLE2_300M = (6912, 768, 6144, 1536, 4608, 3072, 3840, 3840)    # Table 2, 300M x 8 (width 1536)

# Router logit offsets of the skewed-routing stress case: assignment shares ~ rank^-1.2 with rank 1 =
# the widest expert (0.43 of all assignments go to the 8448-wide expert).  Fitted on the seeded train_16k
# tokens with the reference router by tests/golden/fit_router_bias.py; tests/golden/router_bias_zipf.txt
# holds the same numbers with the shares reached.
ZIPF_ROUTER_BIAS = (-2.203125, 0.0, -2.0625, -1.171875, -2.0, -1.53125, -1.8671875, -1.765625)

CONFIGS = {
    "tiny_f32": LayerConfig("tiny_f32", "f32", 64, (96, 160, 112, 144), 2, 256),
    "fwd_8k": LayerConfig("fwd_8k", "bf16", 2048, WIDTHS_700M, 2, 8192, weight_std=0.02, backward=False),
    "train_16k": LayerConfig("train_16k", "bf16", 2048, WIDTHS_700M, 2, 16384, weight_std=0.02),
    "train_16k_equal": LayerConfig("train_16k_equal", "bf16", 2048, WIDTHS_EQUAL, 2, 16384, weight_std=0.02),
    "train_64k": LayerConfig("train_64k", "bf16", 2048, WIDTHS_700M, 2, 65536, weight_std=0.02),
    # size-diversity sweep at a fixed pair sum of 11264 (ratio 1 = train_16k_equal, ratio 3 = train_16k)
    "train_16k_ratio2": LayerConfig("train_16k_ratio2", "bf16", 2048, WIDTHS_RATIO2, 2, 16384, weight_std=0.02),
    "train_16k_ratio4": LayerConfig("train_16k_ratio4", "bf16", 2048, WIDTHS_RATIO4, 2, 16384, weight_std=0.02),
    # the paper's own expert widths (Table 2): ratio 9 at width 2048, and the 300M x 8 model at width 1536
    "table2_700m": LayerConfig("table2_700m", "bf16", 2048, WIDTHS_TABLE2_700M, 2, 16384, weight_std=0.02),
    "table2_300m": LayerConfig("table2_300m", "bf16", 1536, WIDTHS_TABLE2_300M, 2, 16384, weight_std=0.02),
    "train_16k_skew": LayerConfig("train_16k_skew", "bf16", 2048, WIDTHS_700M, 2, 16384, weight_std=0.02,
                                  router_bias=ZIPF_ROUTER_BIAS),
    "train_16k_equal_skew": LayerConfig("train_16k_equal_skew", "bf16", 2048, WIDTHS_EQUAL, 2, 16384,
                                        weight_std=0.02, router_bias=ZIPF_ROUTER_BIAS),
}


def with_tokens(cfg: LayerConfig, n_tokens: int) -> LayerConfig:
    return replace(cfg, n_tokens=n_tokens, name=f"{cfg.name}_T{n_tokens}")


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result is
    float32 holding exactly representable bfloat16 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


@dataclass
class LayerInputs:
    cfg: LayerConfig
    x: np.ndarray            # [T,d] float32 (bf16-representable when cfg.dtype == "bf16")
    w_router: np.ndarray     # [N,d]
    w_gate: list             # N x [h_e,d]
    w_up: list               # N x [h_e,d]
    w_down: list             # N x [d,h_e]
    dy: np.ndarray           # [T,d]
    rng: np.random.Generator = field(repr=False, default=None)

    def redraw_x(self, rng: np.random.Generator, n: int) -> np.ndarray:
        """Fresh token rows with the distribution (and bias channel) of x."""
        rows = to_storage(rng.standard_normal((n, self.cfg.d_model), dtype=np.float32), self.cfg.dtype)
        if self.cfg.router_bias is not None:
            rows[:, -1] = 1.0
        return rows


def generate(cfg: LayerConfig, routing_only: bool = False) -> LayerInputs:
    """Seeded inputs of `cfg`.  With routing_only the expert weights and dY are left out (empty
    lists / None); x and W_router are the first two draws, so they are the same either way."""
    rng = np.random.default_rng(cfg.seed)
    d, N, T = cfg.d_model, cfg.n_experts, cfg.n_tokens

    def normal(shape, std):
        return (rng.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(np.float32)

    def wstd(fan_in):
        return cfg.weight_std if cfg.weight_std is not None else float(fan_in) ** -0.5

    x = normal((T, d), 1.0)
    w_router = normal((N, d), wstd(d))
    if routing_only:
        if cfg.router_bias is not None:
            x[:, -1] = 1.0
            w_router[:, -1] = np.asarray(cfg.router_bias, dtype=np.float32)
        return LayerInputs(cfg, to_storage(x, cfg.dtype), to_storage(w_router, cfg.dtype), [], [], [], None, rng)
    w_gate = [normal((h, d), wstd(d)) for h in cfg.ffn_sizes]
    w_up = [normal((h, d), wstd(d)) for h in cfg.ffn_sizes]
    w_down = [normal((d, h), wstd(h)) for h in cfg.ffn_sizes]
    dy = normal((T, d), 1.0)
    if cfg.router_bias is not None:
        x[:, -1] = 1.0
        w_router[:, -1] = np.asarray(cfg.router_bias, dtype=np.float32)
    s = lambda a: to_storage(a, cfg.dtype)
    return LayerInputs(cfg, s(x), s(w_router), [s(w) for w in w_gate], [s(w) for w in w_up],
                       [s(w) for w in w_down], s(dy), rng)
