"""Pins for the oracle's router (Sec. 2, Eq. 2-3) and permutation bookkeeping."""
import numpy as np
import pytest

from oracle import modse_oracle as O


def _rand(T=200, d=24, N=6, seed=1):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((T, d)), rng.standard_normal((N, d)) / np.sqrt(d)


@pytest.mark.parametrize("k", [1, 2, 3])
def test_topk_matches_full_sort(k):
    x, wr = _rand()
    rt = O.route(x, wr, k)
    z = x @ wr.T                                   # library matmul, independent of the C loops
    np.testing.assert_allclose(rt.z, z, rtol=1e-12, atol=1e-12)
    order = np.argsort(-z, axis=1, kind="stable")[:, :k]     # stable: ties -> lower index
    np.testing.assert_array_equal(rt.topk_idx, order.astype(np.int32))


def test_gates_sum_to_one_and_closed_form():
    x, wr = _rand()
    rt = O.route(x, wr, 2)
    np.testing.assert_allclose(rt.topk_gate.sum(1), 1.0, atol=1e-14)
    z0 = np.take_along_axis(rt.z, rt.topk_idx[:, :1].astype(np.int64), 1)[:, 0]
    z1 = np.take_along_axis(rt.z, rt.topk_idx[:, 1:2].astype(np.int64), 1)[:, 0]
    g0 = 1.0 / (1.0 + np.exp(-(z0 - z1)))         # softmax of two logits = sigmoid of the gap
    np.testing.assert_allclose(rt.topk_gate[:, 0], g0, rtol=1e-13)
    assert np.all(rt.topk_gate[:, 0] >= rt.topk_gate[:, 1])


def test_gates_equal_renormalised_full_softmax():
    # Softmax(KeepTopK(z)) == full softmax restricted to the kept entries and renormalised
    x, wr = _rand(N=7)
    k = 3
    rt = O.route(x, wr, k)
    p = np.exp(rt.z - rt.z.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    kept = np.take_along_axis(p, rt.topk_idx.astype(np.int64), 1)
    np.testing.assert_allclose(rt.topk_gate, kept / kept.sum(1, keepdims=True), rtol=1e-12)


def test_top1_gate_is_one():
    x, wr = _rand()
    rt = O.route(x, wr, 1)
    np.testing.assert_array_equal(rt.topk_gate, np.ones_like(rt.topk_gate))


@pytest.mark.parametrize("k", [1, 2, 3])
def test_permutation_invariants(k):
    x, wr = _rand(T=333)
    T, N = x.shape[0], wr.shape[0]
    rt = O.route(x, wr, k)
    assert rt.counts.sum() == k * T
    np.testing.assert_array_equal(rt.counts, rt.counts_slot.sum(0))
    np.testing.assert_array_equal(rt.counts_slot.sum(1), np.full(k, T))
    np.testing.assert_array_equal(rt.offsets, np.concatenate([[0], np.cumsum(rt.counts)]))
    # bijection onto [0, kT) and inverse map
    np.testing.assert_array_equal(np.sort(rt.row_of.reshape(-1)), np.arange(k * T))
    np.testing.assert_array_equal(rt.token_of[rt.row_of], np.repeat(np.arange(T)[:, None], k, 1))
    # every token appears exactly k times
    np.testing.assert_array_equal(np.bincount(rt.token_of, minlength=T), np.full(T, k))
    # rows sorted by (expert, token): brute-force reconstruction
    pairs = sorted((int(rt.topk_idx[t, j]), t) for t in range(T) for j in range(k))
    np.testing.assert_array_equal(rt.token_of, np.array([p[1] for p in pairs]))
    for e in range(N):
        seg = rt.token_of[rt.offsets[e]:rt.offsets[e + 1]]
        assert np.all(np.diff(seg) > 0)
        for t in seg[:5]:
            assert e in rt.topk_idx[t]


def test_zero_token_and_duplicate_rows_tie_to_lower_index():
    x, wr = _rand(T=8, N=5)
    x[3] = 0.0
    rt = O.route(x, wr, 2)
    np.testing.assert_array_equal(rt.topk_idx[3], [0, 1])
    np.testing.assert_allclose(rt.topk_gate[3], [0.5, 0.5])
    wr2 = wr.copy()
    wr2[4] = wr2[1]                                # experts 1 and 4 always tie exactly
    rt2 = O.route(x, wr2, 2)
    for t in range(8):
        row = list(rt2.topk_idx[t])
        if 4 in row:
            assert 1 in row and row.index(1) < row.index(4)


def test_logit_shift_and_expert_relabelling():
    x, wr = _rand(T=64, d=12, N=5)
    rt = O.route(x, wr, 2)
    # a constant added to every logit of a token changes nothing: append a constant
    # input channel whose router weight is the same for all experts
    x2 = np.concatenate([x, np.ones((64, 1))], 1)
    wr2 = np.concatenate([wr, np.full((5, 1), 3.25)], 1)
    rt2 = O.route(x2, wr2, 2)
    np.testing.assert_array_equal(rt.topk_idx, rt2.topk_idx)
    np.testing.assert_allclose(rt.topk_gate, rt2.topk_gate, rtol=1e-12)
    perm = np.array([3, 0, 4, 1, 2])               # new expert i is old expert perm[i]
    rt3 = O.route(x, wr[perm], 2)
    np.testing.assert_array_equal(perm[rt3.topk_idx], rt.topk_idx)
    np.testing.assert_allclose(rt3.topk_gate, rt.topk_gate, rtol=1e-13)


def test_empty_batch_and_bad_arguments():
    rt = O.route(np.zeros((0, 4)), np.ones((3, 4)), 2)
    np.testing.assert_array_equal(rt.counts, [0, 0, 0])
    np.testing.assert_array_equal(rt.offsets, [0, 0, 0, 0])
    with pytest.raises(RuntimeError):
        O.route(np.zeros((2, 4)), np.ones((3, 4)), 4)         # k > N
    bad = np.zeros((2, 4)); bad[1, 2] = np.inf
    with pytest.raises(RuntimeError):
        O.route(bad, np.ones((3, 4)), 1)


def test_margin_screening_removes_near_ties():
    rng = np.random.default_rng(5)
    T, d, N = 4000, 8, 8
    x = rng.standard_normal((T, d)); wr = rng.standard_normal((N, d))
    before = (O.routing_margin(O.route(x, wr, 2).z, 2) < 1e-3).sum()
    assert before > 0
    xs, n = O.screen_inputs(x, wr, 2, rng, lambda r, m: r.standard_normal((m, d)), tau=1e-3)
    assert n >= before
    assert (O.routing_margin(O.route(xs, wr, 2).z, 2) >= 1e-3).all()


def test_aux_loss_closed_forms():
    # Eq. 7-10: uniform probabilities (all logits equal) give P_i = 1/N and every arg-max
    # goes to expert 0, so L_a = alpha * N * (1 * 1/N) = alpha.
    T, N = 50, 8
    loss, f, P, dz = O.aux_loss(np.zeros((T, N)), 0.01)
    assert abs(loss - 0.01) < 1e-15
    np.testing.assert_allclose(P, 1.0 / N)
    np.testing.assert_array_equal(f, [1.0] + [0.0] * (N - 1))
    # perfectly balanced one-hot routing with huge logits: f_i = P_i = 1/N -> L_a = alpha
    z = np.full((T * N, N), -50.0)
    z[np.arange(T * N), np.arange(T * N) % N] = 50.0
    loss, f, P, _ = O.aux_loss(z, 0.5)
    np.testing.assert_allclose(f, 1.0 / N)
    assert abs(loss - 0.5) < 1e-12
    # gradient (f held fixed) against central differences
    rng = np.random.default_rng(0)
    z = rng.standard_normal((6, 5))
    _, f, _, dz = O.aux_loss(z, 0.3)
    for (t, i) in [(0, 0), (2, 3), (5, 4)]:
        e = np.zeros_like(z); e[t, i] = 1e-6
        Pp = O.aux_loss(z + e, 0.3)[2]; Pm = O.aux_loss(z - e, 0.3)[2]
        num = 0.3 * 5 * np.dot(f, (Pp - Pm)) / 2e-6
        assert abs(num - dz[t, i]) < 1e-8
