"""Pins for the oracle's relational layer (Appendix A), CPU only: the dense matrix form of the layer, closed
forms, reduction to the mean aggregation, and finite differences for both backward passes."""
import numpy as np

import oracle
from helpers import count_matrix, small_problem


def relations(n, sizes, seed):
    """One small random graph per relation (different edge counts, some rows without in-edges)."""
    ps = [small_problem(n, e, 1, 4, seed + 10 * r) for r, e in enumerate(sizes)]
    return ps, [(p["indptr"], p["indices"]) for p in ps]


def test_layer_is_the_sum_of_row_normalised_matrix_products():
    n, d_in, d_out = 40, 6, 5
    ps, graphs = relations(n, (150, 60, 10), 3)
    rng = np.random.default_rng(0)
    h = rng.standard_normal((n, d_in))
    ws = [rng.standard_normal((d_in, d_out)) for _ in graphs]
    want = np.zeros((n, d_out))
    for p, w in zip(ps, ws):
        C = count_matrix(n, n, p["src"], p["dst"]).astype(np.float64)  # C[i, j] = number of edges j -> i
        deg = C.sum(axis=1)
        inv = np.divide(1.0, deg, out=np.zeros_like(deg), where=deg > 0)
        want += (inv[:, None] * C) @ h @ w
    got = oracle.rgcn_layer(graphs, h, ws)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)


def test_identical_features_give_the_sum_of_the_transforms_of_the_relations_present():
    n, d_in, d_out = 30, 4, 3
    ps, graphs = relations(n, (90, 25), 5)
    rng = np.random.default_rng(1)
    x = rng.standard_normal(d_in)
    ws = [rng.standard_normal((d_in, d_out)) for _ in graphs]
    got = oracle.rgcn_layer(graphs, np.tile(x, (n, 1)), ws)
    for i in range(n):
        want = np.zeros(d_out)
        for (indptr, _), w in zip(graphs, ws):
            if indptr[i + 1] > indptr[i]:
                want += x @ w
        assert np.allclose(got[i], want, rtol=1e-12, atol=1e-12)


def test_one_relation_with_the_identity_is_the_mean_aggregation():
    p = small_problem(50, 300, 1, 4, 9)
    rng = np.random.default_rng(2)
    h = rng.standard_normal((50, 4)).astype(np.float32)
    got = oracle.rgcn_layer([(p["indptr"], p["indices"])], h, [np.eye(4)])
    assert np.allclose(got, oracle.spmm(p["indptr"], p["indices"], h, mean=True), rtol=1e-12, atol=1e-12)


def test_backward_matches_finite_differences():
    n, d_in, d_out = 20, 3, 4
    _, graphs = relations(n, (70, 30), 7)
    rng = np.random.default_rng(3)
    h = rng.standard_normal((n, d_in))
    ws = [rng.standard_normal((d_in, d_out)) for _ in graphs]
    gz = rng.standard_normal((n, d_out))
    dh, dws = oracle.rgcn_layer_bwd(graphs, h, ws, gz)
    loss = lambda h_, ws_: float((oracle.rgcn_layer(graphs, h_, ws_) * gz).sum())
    eps = 1e-6
    for (i, k) in [(0, 0), (5, 2), (19, 1), (11, 0)]:
        hp, hm = h.copy(), h.copy()
        hp[i, k] += eps
        hm[i, k] -= eps
        assert abs((loss(hp, ws) - loss(hm, ws)) / (2 * eps) - dh[i, k]) < 1e-7
    for r in range(len(ws)):
        for (k, o) in [(0, 0), (2, 3), (1, 2)]:
            wp = [w.copy() for w in ws]
            wm = [w.copy() for w in ws]
            wp[r][k, o] += eps
            wm[r][k, o] -= eps
            assert abs((loss(h, wp) - loss(h, wm)) / (2 * eps) - dws[r][k, o]) < 1e-7


def test_basis_decomposition_and_its_backward():
    rng = np.random.default_rng(4)
    R, Bn, shape = 4, 2, (3, 5)
    a, V = rng.standard_normal((R, Bn)), rng.standard_normal((Bn,) + shape)
    W = oracle.rgcn_basis(a, V)
    assert np.allclose(W, np.einsum("rb,bxy->rxy", a, V), rtol=1e-13, atol=1e-13)
    onehot = np.zeros((R, Bn))
    onehot[np.arange(R), np.arange(R) % Bn] = 1.0
    assert np.array_equal(oracle.rgcn_basis(onehot, V), V[np.arange(R) % Bn])  # a one-hot row selects its basis tensor
    dW = rng.standard_normal((R,) + shape)
    da, dV = oracle.rgcn_basis_bwd(a, V, dW)
    loss = lambda a_, V_: float((oracle.rgcn_basis(a_, V_) * dW).sum())
    eps = 1e-6
    for (r, b) in [(0, 0), (3, 1), (2, 0)]:
        ap, am = a.copy(), a.copy()
        ap[r, b] += eps
        am[r, b] -= eps
        assert abs((loss(ap, V) - loss(am, V)) / (2 * eps) - da[r, b]) < 1e-7
    for idx in [(0, 0, 0), (1, 2, 4)]:
        Vp, Vm = V.copy(), V.copy()
        Vp[idx] += eps
        Vm[idx] -= eps
        assert abs((loss(a, Vp) - loss(a, Vm)) / (2 * eps) - dV[idx]) < 1e-7
