"""Pins for the oracle's second router term, H(x)_i = (x W_g)_i + RMSNorm(Softplus((x W_n)_i))
(Sec. 2, Eq. 2 with the RMSNorm and Softplus definitions below it): closed forms, the unit-RMS
invariant, finite differences of its own forward, and the chain through the whole layer."""
import math

import numpy as np
import pytest

from oracle import modse_oracle as O
from test_oracle_forward import make


def test_zero_gamma_removes_the_term():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((9, 6)); wn = rng.standard_normal((5, 6))
    r, u = O.noise_term(x, wn, 0.0, 1e-6)
    np.testing.assert_array_equal(r, 0.0)
    np.testing.assert_allclose(u, x @ wn.T, rtol=0, atol=1e-14)


def test_single_entry_closed_form():
    # one expert, x W_n = 0: softplus(0) = ln 2, RMSNorm of a single entry is gamma s / sqrt(s^2 + eps)
    gamma, eps = 0.7, 0.01
    r, u = O.noise_term(np.array([[1.0]]), np.array([[0.0]]), gamma, eps)
    s = math.log(2.0)
    assert u[0, 0] == 0.0
    assert abs(r[0, 0] - gamma * s / math.sqrt(s * s + eps)) < 1e-15


def test_worked_example_three_experts():
    # u = (0, ln(e-1), -40): softplus = (ln 2, 1, ~e^-40)
    u3 = np.array([0.0, math.log(math.e - 1.0), -40.0])
    x = np.array([[1.0, 0.0]]); wn = np.stack([u3, np.zeros(3)], 1)
    gamma, eps = 2.0, 0.0
    r, _ = O.noise_term(x, wn, gamma, eps)
    s = np.array([math.log(2.0), 1.0, math.exp(-40.0)])
    q = math.sqrt((s ** 2).sum() / 3.0)
    np.testing.assert_allclose(r[0], gamma * s / q, rtol=1e-14)


def test_unit_rms_invariant_and_sign():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((40, 12)); wn = rng.standard_normal((8, 12))
    gamma = -1.3
    r, _ = O.noise_term(x, wn, gamma, 0.0)
    np.testing.assert_allclose(np.sqrt((r ** 2).mean(1)), abs(gamma), rtol=1e-13)
    assert (r < 0).all()                                  # softplus > 0, so the sign is gamma's
    # with eps > 0 the RMS is gamma sqrt(ms / (ms + eps)) < |gamma|
    r2, u = O.noise_term(x, wn, gamma, 0.5)
    ms = (np.logaddexp(0.0, u) ** 2).mean(1)
    np.testing.assert_allclose(np.sqrt((r2 ** 2).mean(1)), abs(gamma) * np.sqrt(ms / (ms + 0.5)), rtol=1e-13)


def test_softplus_tails():
    # softplus(u) -> u for large u and -> exp(u) for very negative u, without overflow
    x = np.array([[1.0]]); gamma = 1.0
    for big in (50.0, 800.0):
        r, _ = O.noise_term(x, np.array([[big], [-big]]), gamma, 0.0)
        assert np.isfinite(r).all()
        # s = (big, ~0): q = big / sqrt(2), r = (sqrt 2, ~0)
        assert abs(r[0, 0] - math.sqrt(2.0)) < 1e-12 and 0.0 <= r[0, 1] < 1e-12


def test_term_is_invariant_to_permuting_experts_and_scaling_by_gamma():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((7, 5)); wn = rng.standard_normal((6, 5))
    r, _ = O.noise_term(x, wn, 1.0, 1e-3)
    perm = rng.permutation(6)
    rp, _ = O.noise_term(x, wn[perm], 1.0, 1e-3)
    np.testing.assert_allclose(rp, r[:, perm], rtol=1e-14)
    r3, _ = O.noise_term(x, wn, 3.0, 1e-3)
    np.testing.assert_allclose(r3, 3.0 * r, rtol=1e-14)


@pytest.mark.parametrize("N", [1, 4, 8])
def test_noise_backward_matches_finite_differences(N):
    rng = np.random.default_rng(3 + N)
    T, d = 6, 7
    x = rng.standard_normal((T, d)); wn = rng.standard_normal((N, d)); c = rng.standard_normal((T, N))
    gamma, eps = 0.8, 1e-2

    def L(x_, wn_, g_):
        return float((O.noise_term(x_, wn_, g_, eps)[0] * c).sum())

    dx, dwn, dgamma = O.noise_backward(x, wn, gamma, eps, c)
    h = 1e-6
    for arr, grad, which in ((x, dx, 0), (wn, dwn, 1)):
        for _ in range(10):
            idx = tuple(int(rng.integers(0, s)) for s in arr.shape)
            old = arr[idx]
            arr[idx] = old + h; lp = L(x, wn, gamma)
            arr[idx] = old - h; lm = L(x, wn, gamma)
            arr[idx] = old
            num = (lp - lm) / (2 * h)
            assert abs(num - grad[idx]) <= 1e-7 * max(1.0, abs(num)), (which, idx, num, grad[idx])
    num = (L(x, wn, gamma + h) - L(x, wn, gamma - h)) / (2 * h)
    assert abs(num - dgamma) <= 1e-7 * max(1.0, abs(num))


def test_gradient_vanishes_along_the_scale_direction_when_eps_is_zero():
    # With eps = 0 the term depends on s = softplus(u) only through its direction, so an upstream
    # gradient proportional to s gives ds = 0: nothing reaches x or W_n, and dgamma = sum_t |s_t|^2 / q_t.
    rng = np.random.default_rng(5)
    T, d, N = 5, 4, 6
    x = rng.standard_normal((T, d)); wn = rng.standard_normal((N, d))
    s = np.logaddexp(0.0, x @ wn.T)
    dx, dwn, dgamma = O.noise_backward(x, wn, 1.1, 0.0, s)
    np.testing.assert_allclose(dx, 0.0, atol=1e-12)
    np.testing.assert_allclose(dwn, 0.0, atol=1e-12)
    q = np.sqrt((s ** 2).mean(1))
    assert abs(dgamma - float(((s ** 2).sum(1) / q).sum())) < 1e-10


def test_route_from_logits_agrees_with_route_and_brute_force():
    x, wr, wg, wu, wd = make(T=50, d=9, h=(8, 8, 16, 8, 24), k=2, seed=4)
    rt = O.route(x, wr, 2)
    rt2 = O.route_from_logits(rt.z, 2)
    for name in ("topk_idx", "topk_gate", "counts", "counts_slot", "offsets", "row_of", "token_of"):
        np.testing.assert_array_equal(getattr(rt2, name), getattr(rt, name), err_msg=name)
    # brute force on the logits: stable descending sort, softmax over the kept pair
    order = np.argsort(-rt.z, axis=1, kind="stable")[:, :2]
    np.testing.assert_array_equal(rt2.topk_idx, order)
    kept = np.take_along_axis(rt.z, order, 1)
    w = np.exp(kept - kept.max(1, keepdims=True))
    np.testing.assert_allclose(rt2.topk_gate, w / w.sum(1, keepdims=True), rtol=1e-14)
    # ties go to the lower index
    z = np.array([[1.0, 3.0, 3.0, 0.0], [2.0, 2.0, 2.0, 2.0]])
    np.testing.assert_array_equal(O.route_from_logits(z, 2).topk_idx, [[1, 2], [0, 1]])


def test_layer_gradients_through_the_noise_term():
    """Whole layer with H = x W_g + r: the loss' finite differences in x, W_g, W_n and gamma equal
    backward() (given the noisy routing) plus noise_backward() fed with backward()'s dz."""
    k, T, d = 2, 10, 8
    x, wr, wg, wu, wd = make(T=T, d=d, h=(8, 16, 8, 24), k=k, seed=21)
    rng = np.random.default_rng(77)
    N = wr.shape[0]
    wn = 0.5 * rng.standard_normal((N, d)); gamma, eps = 0.6, 1e-5
    dy = rng.standard_normal((T, d))
    pw = O.pack_weights(wg, wu, wd)

    def logits(x_, wr_, wn_, g_):
        return x_ @ wr_.T + O.noise_term(x_, wn_, g_, eps)[0]

    def L(x_, wr_, wn_, g_):
        rt_ = O.route_from_logits(logits(x_, wr_, wn_, g_), k)
        return float((O.forward_tokens(x_, pw, rt_) * dy).sum())

    # keep only tokens that are far from a routing boundary under the noisy logits
    z = logits(x, wr, wn, gamma)
    keep = O.routing_margin(z, k) > 1e-2
    assert keep.sum() >= 6
    x = np.ascontiguousarray(x[keep]); dy = np.ascontiguousarray(dy[keep])
    rt = O.route_from_logits(logits(x, wr, wn, gamma), k)
    g = O.backward(x, wr, wg, wu, wd, rt, dy)
    dx_add, dwn, dgamma = O.noise_backward(x, wn, gamma, eps, g.dz)
    h = 1e-6
    for arr, grad in ((x, g.dx + dx_add), (wr, g.dw_router), (wn, dwn)):
        for _ in range(12):
            idx = tuple(int(rng.integers(0, s)) for s in arr.shape)
            old = arr[idx]
            arr[idx] = old + h; lp = L(x, wr, wn, gamma)
            arr[idx] = old - h; lm = L(x, wr, wn, gamma)
            arr[idx] = old
            num = (lp - lm) / (2 * h)
            assert abs(num - grad[idx]) <= 2e-6 * max(1.0, abs(num)), (idx, num, grad[idx])
    num = (L(x, wr, wn, gamma + h) - L(x, wr, wn, gamma - h)) / (2 * h)
    assert abs(num - dgamma) <= 2e-6 * max(1.0, abs(num))


def test_planted_mistakes_are_caught():
    """The pins above separate the definition from near misses: RMS over the wrong axis, a dropped
    1/N, sigmoid forgotten in the chain rule."""
    rng = np.random.default_rng(8)
    x = rng.standard_normal((6, 5)); wn = rng.standard_normal((4, 5))
    r, u = O.noise_term(x, wn, 1.0, 0.0)
    s = np.logaddexp(0.0, u)
    wrong_axis = s / np.sqrt((s ** 2).mean(0, keepdims=True))
    no_mean = s / np.sqrt((s ** 2).sum(1, keepdims=True))
    assert np.abs(r - wrong_axis).max() > 1e-3 and np.abs(r - no_mean).max() > 1e-3
    c = rng.standard_normal(r.shape)
    dx, dwn, _ = O.noise_backward(x, wn, 1.0, 0.0, c)
    q = np.sqrt((s ** 2).mean(1, keepdims=True))
    ds = c / q - s * (c * s).sum(1, keepdims=True) / (4 * q ** 3)
    no_sigmoid = ds.T @ x
    assert np.abs(dwn - no_sigmoid).max() > 1e-3
