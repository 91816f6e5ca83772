"""numpy front end of the fp64 C oracle of the MoDSE layer.

Test infrastructure only: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the CUDA product path.  Every function
marshals arguments to ``libmodse_oracle.so``; the arithmetic is in
``modse_oracle.c`` and follows Sec. 2 (Eq. 1-3), Sec. 3.1 (Eq. 4-6) and
Sec. 3.2 (Eq. 7-10) of the paper.

Weights are passed as per-expert lists: ``w_gate[e], w_up[e]`` of shape
``[h_e, d]`` and ``w_down[e]`` of shape ``[d, h_e]``.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from . import build as _build

_lib = None
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.modse_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().modse_oracle_num_threads())


def _d(a):
    return None if a is None else a.ctypes.data_as(_D)


def _i(a):
    return None if a is None else a.ctypes.data_as(_I)


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _check(rc: int, what: str):
    if rc != 0:
        reason = {-1: "bad argument", -2: "non-finite router logit", -3: "out of memory"}.get(rc, "?")
        raise RuntimeError(f"oracle {what} failed: {rc} ({reason})")


@dataclass
class Routing:
    z: np.ndarray            # [T,N] router logits
    topk_idx: np.ndarray     # [T,k] int32, slot 0 = largest
    topk_gate: np.ndarray    # [T,k]
    counts: np.ndarray       # [N]
    counts_slot: np.ndarray  # [k,N]
    offsets: np.ndarray      # [N+1]
    row_of: np.ndarray       # [T,k]
    token_of: np.ndarray     # [k*T]


@dataclass
class PackedWeights:
    h: np.ndarray        # [N] int32
    w_gate: np.ndarray   # [S,d]
    w_up: np.ndarray     # [S,d]
    w_down: np.ndarray   # flat, expert e = [d,h_e] block at d*off_e


def pack_weights(w_gate, w_up, w_down) -> PackedWeights:
    h = _i32([w.shape[0] for w in w_gate])
    return PackedWeights(
        h=h,
        w_gate=_f64(np.concatenate([_f64(w) for w in w_gate], axis=0)),
        w_up=_f64(np.concatenate([_f64(w) for w in w_up], axis=0)),
        w_down=_f64(np.concatenate([_f64(w).reshape(-1) for w in w_down])),
    )


def unpack_like(pw: PackedWeights, d: int, flat_gate, flat_up, flat_down):
    """Split packed gradient arrays back into per-expert lists."""
    g, u, dn = [], [], []
    off = 0
    for he in pw.h:
        he = int(he)
        g.append(flat_gate[off:off + he])
        u.append(flat_up[off:off + he])
        dn.append(flat_down[d * off:d * (off + he)].reshape(d, he))
        off += he
    return g, u, dn


def route(x, w_router, k: int) -> Routing:
    x = _f64(x); w_router = _f64(w_router)
    T, d = x.shape
    N = w_router.shape[0]
    z = np.empty((T, N)); idx = np.empty((T, k), np.int32); gate = np.empty((T, k))
    counts = np.empty(N, np.int32); cs = np.empty((k, N), np.int32)
    offsets = np.empty(N + 1, np.int32); row_of = np.empty((T, k), np.int32)
    token_of = np.empty(k * T, np.int32)
    rc = lib().modse_oracle_route(T, d, N, k, _d(x), _d(w_router), _d(z), _i(idx), _d(gate),
                                  _i(counts), _i(cs), _i(offsets), _i(row_of), _i(token_of))
    _check(rc, "route")
    return Routing(z, idx, gate, counts, cs, offsets, row_of, token_of)


def forward_tokens(x, pw: PackedWeights, rt: Routing, sel=None, want_o=False):
    x = _f64(x)
    T, d = x.shape
    N = len(pw.h); k = rt.topk_idx.shape[1]
    sel_a = _i32(np.arange(T) if sel is None else sel)
    n = len(sel_a)
    y = np.empty((n, d)); o = np.empty((n, k, d)) if want_o else None
    rc = lib().modse_oracle_forward_tokens(T, d, N, k, _i(pw.h), _d(x), _d(pw.w_gate), _d(pw.w_up),
                                           _d(pw.w_down), _i(rt.topk_idx), _d(rt.topk_gate),
                                           n, _i(sel_a), _d(y), _d(o))
    _check(rc, "forward_tokens")
    return (y, o) if want_o else y


def forward(x, w_router, w_gate, w_up, w_down, k: int):
    """Whole layer: returns (y [T,d], Routing)."""
    rt = route(x, w_router, k)
    pw = pack_weights(w_gate, w_up, w_down)
    return forward_tokens(x, pw, rt), rt


def backward_tokens(x, w_router, pw: PackedWeights, rt: Routing, dy, sel=None):
    """(dx_sel, dg_sel, dz_sel) for the listed tokens."""
    x = _f64(x); dy = _f64(dy); w_router = _f64(w_router)
    T, d = x.shape
    N = len(pw.h); k = rt.topk_idx.shape[1]
    sel_a = _i32(np.arange(T) if sel is None else sel)
    n = len(sel_a)
    dx = np.empty((n, d)); dg = np.empty((n, k)); dz = np.empty((n, N))
    rc = lib().modse_oracle_backward_tokens(T, d, N, k, _i(pw.h), _d(x), _d(w_router), _d(pw.w_gate),
                                            _d(pw.w_up), _d(pw.w_down), _i(rt.topk_idx), _d(rt.topk_gate),
                                            _d(dy), n, _i(sel_a), _d(dx), _d(dg), _d(dz))
    _check(rc, "backward_tokens")
    return dx, dg, dz


def wgrad_rows(x, pw: PackedWeights, rt: Routing, dy, rows_e, rows_r):
    """(dW_gate rows, dW_up rows, dW_down columns), each [n_rows, d]."""
    x = _f64(x); dy = _f64(dy)
    T, d = x.shape
    N = len(pw.h); k = rt.topk_idx.shape[1]
    re_, rr_ = _i32(rows_e), _i32(rows_r)
    n = len(re_)
    a = np.empty((n, d)); b = np.empty((n, d)); c = np.empty((n, d))
    rc = lib().modse_oracle_wgrad_rows(T, d, N, k, _i(pw.h), _d(x), _d(pw.w_gate), _d(pw.w_up), _d(pw.w_down),
                                       _i(rt.topk_idx), _d(rt.topk_gate), _d(dy), n, _i(re_), _i(rr_),
                                       _d(a), _d(b), _d(c))
    _check(rc, "wgrad_rows")
    return a, b, c


@dataclass
class Grads:
    dx: np.ndarray
    dw_router: np.ndarray
    dw_gate: list
    dw_up: list
    dw_down: list
    dg: np.ndarray
    dz: np.ndarray


def backward(x, w_router, w_gate, w_up, w_down, rt: Routing, dy) -> Grads:
    x = _f64(x); dy = _f64(dy); w_router = _f64(w_router)
    T, d = x.shape
    pw = pack_weights(w_gate, w_up, w_down)
    N = len(pw.h); k = rt.topk_idx.shape[1]
    S = int(pw.h.sum())
    dx = np.empty((T, d)); dwr = np.empty((N, d))
    dwg = np.empty((S, d)); dwu = np.empty((S, d)); dwd = np.empty(S * d)
    dg = np.empty((T, k)); dz = np.empty((T, N))
    rc = lib().modse_oracle_backward(T, d, N, k, _i(pw.h), _d(x), _d(w_router), _d(pw.w_gate), _d(pw.w_up),
                                     _d(pw.w_down), _i(rt.topk_idx), _d(rt.topk_gate), _d(dy),
                                     _d(dx), _d(dwr), _d(dwg), _d(dwu), _d(dwd), _d(dg), _d(dz))
    _check(rc, "backward")
    g, u, dn = unpack_like(pw, d, dwg, dwu, dwd)
    return Grads(dx, dwr, g, u, dn, dg, dz)


def aux_loss(z, alpha: float):
    """(L_a, f [N], P [N], dL_a/dz [T,N]) of Eq. 7-10."""
    z = _f64(z)
    T, N = z.shape
    loss = ctypes.c_double(0.0)
    f = np.empty(N); P = np.empty(N); dz = np.empty((T, N))
    rc = lib().modse_oracle_aux_loss(T, N, _d(z), ctypes.c_double(alpha), ctypes.byref(loss), _d(f), _d(P), _d(dz))
    _check(rc, "aux_loss")
    return loss.value, f, P, dz


def noise_term(x, w_noise, gamma: float, eps: float):
    """(r [T,N], u [T,N]): r = RMSNorm(Softplus(x W_n)) over the expert entries, u = x W_n."""
    x = _f64(x); w_noise = _f64(w_noise)
    T, d = x.shape
    N = w_noise.shape[0]
    r = np.empty((T, N)); u = np.empty((T, N))
    rc = lib().modse_oracle_noise_term(T, d, N, _d(x), _d(w_noise), ctypes.c_double(gamma), ctypes.c_double(eps),
                                       _d(r), _d(u))
    _check(rc, "noise_term")
    return r, u


def noise_backward(x, w_noise, gamma: float, eps: float, dz):
    """(dx_add [T,d], dw_noise [N,d], dgamma) for dz = dL/dH [T,N]."""
    x = _f64(x); w_noise = _f64(w_noise); dz = _f64(dz)
    T, d = x.shape
    N = w_noise.shape[0]
    dx = np.empty((T, d)); dw = np.empty((N, d)); dg = ctypes.c_double(0.0)
    rc = lib().modse_oracle_noise_backward(T, d, N, _d(x), _d(w_noise), ctypes.c_double(gamma),
                                           ctypes.c_double(eps), _d(dz), _d(dx), _d(dw), ctypes.byref(dg))
    _check(rc, "noise_backward")
    return dx, dw, dg.value


def route_from_logits(z, k: int) -> Routing:
    z = _f64(z)
    T, N = z.shape
    idx = np.empty((T, k), np.int32); gate = np.empty((T, k))
    counts = np.empty(N, np.int32); cs = np.empty((k, N), np.int32)
    offsets = np.empty(N + 1, np.int32); row_of = np.empty((T, k), np.int32)
    token_of = np.empty(k * T, np.int32)
    rc = lib().modse_oracle_route_from_logits(T, N, k, _d(z), _i(idx), _d(gate), _i(counts), _i(cs), _i(offsets),
                                              _i(row_of), _i(token_of))
    _check(rc, "route_from_logits")
    return Routing(z, idx, gate, counts, cs, offsets, row_of, token_of)


def routing_margin(z: np.ndarray, k: int) -> np.ndarray:
    """Smallest gap between consecutive logits among the k+1 largest of each
    token: the distance of the top-k decision (and its order) from a flip."""
    zs = -np.sort(-z, axis=1)
    kk = min(k + 1, z.shape[1])
    if kk < 2:
        return np.full(z.shape[0], np.inf)
    return np.min(zs[:, :kk - 1] - zs[:, 1:kk], axis=1)


def screen_inputs(x, w_router, k: int, rng: np.random.Generator, redraw, tau: float = 1e-4,
                  max_rounds: int = 20):
    """Re-draw (with ``redraw(rng, n) -> [n,d]``) every token whose routing
    margin is below ``tau`` but not exactly zero, so that an fp32-accumulating
    router and this fp64 one cannot legitimately disagree on a near-tie.
    Returns (x_screened, number_of_redrawn_tokens)."""
    x = np.array(x, copy=True)
    total = 0
    for _ in range(max_rounds):
        m = routing_margin(route(x, w_router, k).z, k)
        bad = np.nonzero((m < tau) & (m != 0.0))[0]
        if len(bad) == 0:
            return x, total
        x[bad] = redraw(rng, len(bad))
        total += len(bad)
    raise RuntimeError("margin screening did not converge")
