"""Pins for the oracle's GraphSage layer (Eq. 2), CPU only: dense matrix form, reduction to the mean
aggregation, a closed form, finite differences for the backward pass."""
import numpy as np

import oracle
from helpers import count_matrix, small_problem


def _setup(n, e, d_in, d_out, seed, empty_rows=0):
    p = small_problem(n, e, 1, 4, seed, empty_rows=empty_rows)
    rng = np.random.default_rng(seed)
    return p, rng.standard_normal((n, d_in)), rng.standard_normal((d_in, d_out)), rng.standard_normal((d_in, d_out))


def test_layer_is_the_row_normalised_matrix_product_plus_the_residual_term():
    p, h, w, w_res = _setup(50, 260, 6, 4, 1, empty_rows=3)
    C = count_matrix(50, 50, p["src"], p["dst"])
    deg = C.sum(axis=1)
    inv = np.divide(1.0, deg, out=np.zeros_like(deg), where=deg > 0)
    want = h @ w_res + (inv[:, None] * C) @ (h @ w)
    assert (deg == 0).any()
    assert np.allclose(oracle.sage_layer(p["indptr"], p["indices"], h, w, w_res), want, rtol=1e-12, atol=1e-12)


def test_without_residual_and_with_the_identity_it_is_the_mean_aggregation():
    p, h, _, _ = _setup(40, 200, 5, 5, 2)
    got = oracle.sage_layer(p["indptr"], p["indices"], h, np.eye(5), np.zeros((5, 5)))
    assert np.allclose(got, oracle.spmm(p["indptr"], p["indices"], h.astype(np.float32), mean=True), rtol=1e-6, atol=1e-6)


def test_identical_features_closed_form():
    p, _, w, w_res = _setup(30, 100, 4, 3, 3, empty_rows=2)
    x = np.random.default_rng(9).standard_normal(4)
    got = oracle.sage_layer(p["indptr"], p["indices"], np.tile(x, (30, 1)), w, w_res)
    deg = np.diff(p["indptr"])
    for i in range(30):
        want = x @ w_res + (x @ w if deg[i] else 0.0)
        assert np.allclose(got[i], want, rtol=1e-12, atol=1e-12)


def test_backward_matches_finite_differences():
    p, h, w, w_res = _setup(25, 90, 3, 4, 4, empty_rows=1)
    g = np.random.default_rng(5).standard_normal((25, 4))
    dh, dw, dw_res = oracle.sage_layer_bwd(p["indptr"], p["indices"], h, w, w_res, g)
    loss = lambda h_, w_, r_: float((oracle.sage_layer(p["indptr"], p["indices"], h_, w_, r_) * g).sum())
    eps = 1e-6

    def fd(arrs, which, idx):
        plus = [a.copy() for a in arrs]
        minus = [a.copy() for a in arrs]
        plus[which][idx] += eps
        minus[which][idx] -= eps
        return (loss(*plus) - loss(*minus)) / (2 * eps)

    for idx in [(0, 0), (7, 2), (24, 1)]:
        assert abs(fd([h, w, w_res], 0, idx) - dh[idx]) < 1e-7
    for idx in [(0, 0), (2, 3), (1, 1)]:
        assert abs(fd([h, w, w_res], 1, idx) - dw[idx]) < 1e-7
        assert abs(fd([h, w, w_res], 2, idx) - dw_res[idx]) < 1e-7
