"""Pins for the oracle's gradients: central finite differences of its own forward,
softmax-Jacobian identities, and agreement of the per-sample entry points."""
import numpy as np
import pytest

from oracle import modse_oracle as O
from test_oracle_forward import make


def loss(x, wr, wg, wu, wd, k, dy):
    y, _ = O.forward(x, wr, wg, wu, wd, k)
    return float((y * dy).sum())


def setup(k=2, seed=11, h=(8, 24, 16, 16), T=12, d=10):
    x, wr, wg, wu, wd = make(T=T, d=d, h=h, k=k, seed=seed)
    rng = np.random.default_rng(seed + 100)
    # keep every token far from a routing boundary so a perturbation cannot cross it
    x, _ = O.screen_inputs(x, wr, k, rng, lambda r, n: r.standard_normal((n, d)), tau=1e-2)
    dy = rng.standard_normal((T, d))
    return x, wr, wg, wu, wd, dy


@pytest.mark.parametrize("k", [1, 2, 3])
def test_gradients_match_finite_differences(k):
    x, wr, wg, wu, wd, dy = setup(k=k)
    rt = O.route(x, wr, k)
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    rng = np.random.default_rng(0)
    eps = 1e-6

    def fd(arr, idx):
        old = arr[idx]
        arr[idx] = old + eps; lp = loss(x, wr, wg, wu, wd, k, dy)
        arr[idx] = old - eps; lm = loss(x, wr, wg, wu, wd, k, dy)
        arr[idx] = old
        return (lp - lm) / (2 * eps)

    def check(arr, grad, n=6):
        for _ in range(n):
            idx = tuple(int(rng.integers(0, s)) for s in arr.shape)
            num = fd(arr, idx)
            assert abs(num - grad[idx]) <= 1e-6 * max(1.0, abs(num)), (idx, num, grad[idx])

    check(x, g.dx, 12)
    check(wr, g.dw_router, 12)
    for e in range(len(wg)):
        if rt.counts[e] == 0:
            continue
        check(wg[e], g.dw_gate[e]); check(wu[e], g.dw_up[e]); check(wd[e], g.dw_down[e])


def test_router_gradient_identities():
    x, wr, wg, wu, wd, dy = setup(k=2)
    rt = O.route(x, wr, 2)
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    np.testing.assert_allclose(g.dz.sum(1), 0.0, atol=1e-13)          # Jacobian annihilates constants
    unsel = np.ones_like(g.dz, bool)
    np.put_along_axis(unsel, rt.topk_idx.astype(np.int64), False, 1)
    np.testing.assert_array_equal(g.dz[unsel], 0.0)
    np.testing.assert_allclose(g.dw_router, g.dz.T @ x, rtol=1e-12, atol=1e-13)
    # top-1: gate is the constant 1, so the router receives no gradient
    rt1 = O.route(x, wr, 1)
    g1 = O.backward(x, wr, wg, wu, wd, rt1, dy)
    np.testing.assert_array_equal(g1.dw_router, 0.0)
    np.testing.assert_array_equal(g1.dz, 0.0)


def test_gate_gradient_is_rowdot_of_down_dgrad_with_hidden():
    # dg = <dY, W_down hm> = <W_down^T dY, hm>
    x, wr, wg, wu, wd, dy = setup(k=2)
    rt = O.route(x, wr, 2)
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    for t in range(x.shape[0]):
        for j in range(2):
            e = rt.topk_idx[t, j]
            a = wg[e] @ x[t]; b = wu[e] @ x[t]
            hm = a / (1 + np.exp(-a)) * b
            assert abs((wd[e].T @ dy[t]) @ hm - g.dg[t, j]) < 1e-12


def test_empty_expert_gets_zero_weight_gradients():
    x, wr, wg, wu, wd, dy = setup(k=2)
    wr = wr.copy(); wr[2] = 0.0; x = np.abs(x); wr[[0, 1, 3]] = np.abs(wr[[0, 1, 3]]) + 0.1
    rt = O.route(x, wr, 2)
    assert rt.counts[2] == 0
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    for arr in (g.dw_gate[2], g.dw_up[2], g.dw_down[2]):
        np.testing.assert_array_equal(arr, 0.0)


def test_sampled_entry_points_agree_with_full_backward():
    x, wr, wg, wu, wd, dy = setup(k=2, T=30)
    rt = O.route(x, wr, 2)
    pw = O.pack_weights(wg, wu, wd)
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    sel = np.array([29, 3, 3, 17], np.int32)
    dx, dg, dz = O.backward_tokens(x, wr, pw, rt, dy, sel)
    np.testing.assert_allclose(dx, g.dx[sel], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dg, g.dg[sel], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dz, g.dz[sel], rtol=1e-12, atol=1e-13)
    rows_e = np.array([0, 1, 1, 3], np.int32); rows_r = np.array([7, 0, 23, 5], np.int32)
    a, b, c = O.wgrad_rows(x, pw, rt, dy, rows_e, rows_r)
    for s, (e, r) in enumerate(zip(rows_e, rows_r)):
        np.testing.assert_allclose(a[s], g.dw_gate[e][r], rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(b[s], g.dw_up[e][r], rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(c[s], g.dw_down[e][:, r], rtol=1e-11, atol=1e-13)
