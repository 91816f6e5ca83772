"""Pins for the oracle's forward values (Eq. 1 and Eq. 4; SwiGLU experts)."""
import os

import numpy as np
import pytest
import torch

from oracle import modse_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table2_expert_widths.txt")


def make(T=40, d=12, h=(8, 24, 16, 16), k=2, seed=3):
    rng = np.random.default_rng(seed)
    N = len(h)
    x = rng.standard_normal((T, d))
    wr = rng.standard_normal((N, d)) / np.sqrt(d)
    wg = [rng.standard_normal((he, d)) / np.sqrt(d) for he in h]
    wu = [rng.standard_normal((he, d)) / np.sqrt(d) for he in h]
    wd = [rng.standard_normal((d, he)) / np.sqrt(he) for he in h]
    return x, wr, wg, wu, wd


def dense_mask_layer(x, wr, wg, wu, wd, k):
    """Eq. 1 literally: every expert on every token, weighted by the full gate
    vector G(x) = Softmax(KeepTopK(H(x), k)) with -inf outside the top-k.
    Written with library routines only (torch fp64), independent of the C code."""
    X = torch.from_numpy(x)
    z = X @ torch.from_numpy(wr).T
    N = z.shape[1]
    keep = torch.full_like(z, float("-inf"))
    zz = z.clone()
    for _ in range(k):                               # k picks, lowest index wins ties
        m = zz.max(dim=1, keepdim=True).values
        first = ((zz == m).float().cumsum(1) == 1) & (zz == m)
        keep[first] = z[first]
        zz[first] = float("-inf")
    G = torch.softmax(keep, dim=1)
    y = torch.zeros_like(X)
    for i in range(N):
        a = X @ torch.from_numpy(wg[i]).T
        b = X @ torch.from_numpy(wu[i]).T
        y += G[:, i:i + 1] * ((torch.nn.functional.silu(a) * b) @ torch.from_numpy(wd[i]).T)
    return y.numpy(), G.numpy()


@pytest.mark.parametrize("k", [1, 2, 3])
def test_matches_dense_mask_form_of_eq1(k):
    x, wr, wg, wu, wd = make()
    y, rt = O.forward(x, wr, wg, wu, wd, k)
    yref, G = dense_mask_layer(x, wr, wg, wu, wd, k)
    np.testing.assert_allclose(y, yref, rtol=1e-11, atol=1e-12)
    Gor = np.zeros_like(G)
    np.put_along_axis(Gor, rt.topk_idx.astype(np.int64), rt.topk_gate, 1)
    np.testing.assert_allclose(Gor, G, rtol=1e-12, atol=1e-15)


def test_single_expert_top1_is_dense_swiglu_ffn():
    x, wr, wg, wu, wd = make(h=(20,), k=1)
    y, rt = O.forward(x, wr, wg, wu, wd, 1)
    X = torch.from_numpy(x)
    ref = (torch.nn.functional.silu(X @ torch.from_numpy(wg[0]).T) * (X @ torch.from_numpy(wu[0]).T)) \
        @ torch.from_numpy(wd[0]).T
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(rt.topk_idx, 0)


def test_equal_width_experts_is_standard_top2_moe():
    x, wr, wg, wu, wd = make(h=(16, 16, 16, 16))
    y, rt = O.forward(x, wr, wg, wu, wd, 2)
    X = torch.from_numpy(x)
    probs = torch.softmax(X @ torch.from_numpy(wr).T, dim=1)          # softmax first ...
    top_p, top_i = torch.topk(probs, 2, dim=1)
    top_p = top_p / top_p.sum(1, keepdim=True)                        # ... then renormalise
    ref = torch.zeros_like(X)
    for e in range(4):                                                # per-expert masked loop
        for j in range(2):
            m = top_i[:, j] == e
            if m.any():
                xe = X[m]
                oe = (torch.nn.functional.silu(xe @ torch.from_numpy(wg[e]).T)
                      * (xe @ torch.from_numpy(wu[e]).T)) @ torch.from_numpy(wd[e]).T
                ref[m] += top_p[m, j:j + 1] * oe
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_array_equal(rt.topk_idx, top_i.numpy().astype(np.int32))


def test_linearity_in_down_projection_and_slot_isolation():
    x, wr, wg, wu, wd = make()
    rt = O.route(x, wr, 2)
    pw = O.pack_weights(wg, wu, wd)
    y, o = O.forward_tokens(x, pw, rt, want_o=True)
    np.testing.assert_allclose(y, (rt.topk_gate[:, :, None] * o).sum(1), rtol=1e-13, atol=1e-14)
    e = 1
    wd2 = [w.copy() for w in wd]; wd2[e] *= 2.5
    y2, o2 = O.forward_tokens(x, O.pack_weights(wg, wu, wd2), rt, want_o=True)
    scale = np.where(rt.topk_idx == e, 2.5, 1.0)[:, :, None]
    np.testing.assert_allclose(o2, o * scale, rtol=1e-13, atol=1e-14)
    wd3 = [w.copy() for w in wd]; wd3[e][:] = 0.0
    y3 = O.forward_tokens(x, O.pack_weights(wg, wu, wd3), rt)
    keep = np.where(rt.topk_idx == e, 0.0, rt.topk_gate)[:, :, None]
    np.testing.assert_allclose(y3, (keep * o).sum(1), rtol=1e-13, atol=1e-14)


def test_zero_token_gives_zero_output_and_subset_mode_agrees():
    x, wr, wg, wu, wd = make()
    x[7] = 0.0
    y, rt = O.forward(x, wr, wg, wu, wd, 2)
    np.testing.assert_array_equal(y[7], 0.0)
    sel = np.array([31, 7, 0, 12], np.int32)
    ysel = O.forward_tokens(x, O.pack_weights(wg, wu, wd), rt, sel=sel)
    np.testing.assert_array_equal(ysel, y[sel])


def test_swiglu_uses_gate_matrix_inside_silu():
    # a transposed/rolled operand must fail: with W_up = 0 the output is 0, with W_gate = 0 too
    x, wr, wg, wu, wd = make(h=(8,), k=1)
    y0, _ = O.forward(x, wr, wg, [np.zeros_like(wu[0])], wd, 1)
    np.testing.assert_array_equal(y0, 0.0)
    # silu(a)*b with a<->b swapped differs: check one scalar case by hand
    # d=1,h=1: a = 2*1, b = 3*1, silu(2)*3 * wd
    y1, _ = O.forward(np.array([[1.0]]), np.array([[1.0]]), [np.array([[2.0]])], [np.array([[3.0]])],
                      [np.array([[0.5]])], 1)
    assert abs(y1[0, 0] - (2.0 / (1.0 + np.exp(-2.0))) * 3.0 * 0.5) < 1e-15


def test_table2_pairs_keep_total_width():
    # Sec. 3.1 Eq. 5-6: each pair sums to 2h, so the total equals N*h of the equal-size model
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    for r in rows:
        if r[0] == "ratios":
            ratios = [float(v) for v in r[1:]]
            continue
    for r in rows:
        if r[0] == "ratios":
            continue
        dm, h = int(r[1]), int(r[2])
        widths = [int(v) for v in r[3:]]
        assert len(widths) == 8
        for p in range(4):
            assert widths[2 * p] + widths[2 * p + 1] == 2 * h
            assert widths[2 * p] >= h >= widths[2 * p + 1]
        assert sum(widths) == 8 * h
        assert [w / dm for w in widths] == ratios
