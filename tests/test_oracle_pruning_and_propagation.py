"""Pins for the oracle's message-flow pruning (Appendix B) and weighted propagation, CPU only: dense formulations, the
definition by reachability, and the invariance it exists for (pruned and full stacks agree on the
labelled nodes)."""
import numpy as np

import oracle
from helpers import count_matrix, small_problem


def test_frontier_is_the_boolean_matrix_product():
    p = small_problem(60, 240, 1, 4, 3)
    rng = np.random.default_rng(0)
    C = count_matrix(60, 60, p["src"], p["dst"]) > 0  # C[i, j]: some edge j -> i
    for density in (0.0, 0.05, 0.3, 1.0):
        need_out = rng.random(60) < density
        want = need_out | (C.T.astype(np.int64) @ need_out.astype(np.int64) > 0)
        got = oracle.mfg_frontier(p["indptr"], p["indices"], need_out)
        assert np.array_equal(got.astype(bool), want)


def test_repeated_frontier_is_bounded_reachability():
    # nodes whose layer-0 input matters for a 3-layer stack = nodes with a directed walk of length <= 3 to a labelled node
    p = small_problem(50, 120, 1, 4, 5)
    A = (count_matrix(50, 50, p["src"], p["dst"]) > 0).astype(np.int64)  # A[i, j]: j -> i
    labelled = np.zeros(50, dtype=bool)
    labelled[[3, 17]] = True
    need = labelled
    for _ in range(3):
        need = oracle.mfg_frontier(p["indptr"], p["indices"], need).astype(bool)
    reach = np.eye(50, dtype=np.int64)
    total = reach.copy()
    for _ in range(3):
        reach = (reach @ A > 0).astype(np.int64)  # reach[i, j]: walk j -> ... -> i of this length
        total = ((total + reach) > 0).astype(np.int64)
    want = total[labelled].sum(axis=0) > 0
    assert np.array_equal(need, want)


def test_filter_rows_keeps_slices_and_empties_the_rest():
    p = small_problem(40, 300, 1, 4, 7, self_loops=True)
    keep = np.arange(40) % 3 != 0
    ptr, idx = oracle.csr_filter_rows(p["indptr"], p["indices"], keep)
    assert ptr[0] == 0 and ptr[-1] == idx.shape[0]
    for i in range(40):
        row = idx[ptr[i]:ptr[i + 1]]
        if keep[i]:
            assert np.array_equal(row, p["indices"][p["indptr"][i]:p["indptr"][i + 1]])
        else:
            assert row.shape[0] == 0
    # as an edge multiset: exactly the edges whose destination is kept
    dst_of = np.repeat(np.arange(40), np.diff(p["indptr"]))
    assert idx.shape[0] == int(keep[dst_of].sum())


def test_pruned_stack_agrees_with_the_full_stack_on_the_labelled_nodes():
    p = small_problem(80, 400, 2, 4, 11)
    rng = np.random.default_rng(2)
    L = 2
    a_l = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    a_r = [rng.standard_normal((2, 4)) * 0.5 for _ in range(L)]
    labelled = np.zeros(80, dtype=bool)
    labelled[[5, 40, 41]] = True

    def stack(graphs):
        z = p["feat"].astype(np.float64)
        for l in range(L):
            ptr, idx = graphs[l]
            el, er = oracle.project(z, a_l[l], a_r[l])
            z = np.maximum(oracle.gat_fwd(ptr, idx, z.astype(np.float32), el.astype(np.float32), er.astype(np.float32), 0.2).out, 0.0)
        return z

    full = stack([(p["indptr"], p["indices"])] * L)
    need = labelled
    graphs = [None] * L
    for l in reversed(range(L)):
        graphs[l] = oracle.csr_filter_rows(p["indptr"], p["indices"], need)
        need = oracle.mfg_frontier(p["indptr"], p["indices"], need).astype(bool)
    pruned = stack(graphs)
    assert np.array_equal(pruned[labelled], full[labelled])
    assert sum(g[1].shape[0] for g in graphs) < L * p["indices"].shape[0]


def test_scaled_sum_is_the_sparse_matrix_product():
    import scipy.sparse as sp
    p = small_problem(70, 500, 1, 6, 17, self_loops=True, empty_rows=3)
    rng = np.random.default_rng(3)
    x = rng.standard_normal((70, 6))
    s_src, s_dst = rng.random(70) + 0.5, rng.random(70) + 0.5
    A = sp.csr_matrix((np.ones(len(p["indices"])), p["indices"], p["indptr"]), shape=(70, 70))  # duplicates add up
    want = sp.diags(s_dst) @ (A @ (sp.diags(s_src) @ x))
    assert np.allclose(oracle.spmm_scaled(p["indptr"], p["indices"], x, s_src, s_dst), want, rtol=1e-13, atol=1e-13)
    assert np.allclose(oracle.spmm_scaled(p["indptr"], p["indices"], x), A @ x, rtol=1e-13, atol=1e-13)
    # symmetric normalisation of an undirected graph: the constant vector d^(1/2) is a fixed point
    src = np.concatenate([p["src"], p["dst"]])
    dst = np.concatenate([p["dst"], p["src"]])
    ptr, idx = oracle.csr_from_coo(70, 70, src, dst)
    deg = np.diff(ptr).astype(np.float64)
    s = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0)
    v = np.sqrt(deg)[:, None]
    assert np.allclose(oracle.spmm_scaled(ptr, idx, v, s, s), v, rtol=1e-12, atol=1e-12)


def _undirected(n, e, seed):
    p = small_problem(n, e, 1, 4, seed)
    src = np.concatenate([p["src"], p["dst"]]).astype(np.int32)
    dst = np.concatenate([p["dst"], p["src"]]).astype(np.int32)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    A = count_matrix(n, n, src, dst)
    deg = A.sum(axis=1)
    inv_sqrt = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0)
    return indptr, indices, A, inv_sqrt


def test_iterated_propagation_steps_and_fixed_point():
    n, alpha = 45, 0.8
    indptr, indices, A, s = _undirected(n, 120, 13)
    S = s[:, None] * A * s[None, :]
    x0 = np.random.default_rng(3).standard_normal((n, 3))
    assert np.array_equal(oracle.propagate(indptr, indices, x0, alpha, 0, s, s), x0)
    one = oracle.propagate(indptr, indices, x0, alpha, 1, s, s)
    assert np.allclose(one, (1 - alpha) * x0 + alpha * S @ x0, rtol=1e-13, atol=1e-13)
    two = oracle.propagate(indptr, indices, x0, alpha, 2, s, s)
    assert np.allclose(two, (1 - alpha) * x0 + alpha * S @ one, rtol=1e-13, atol=1e-13)
    # the eigenvalues of the symmetric normalisation lie in [-1, 1]: the iteration converges to (1-a)(I - aS)^-1 x0
    limit = np.linalg.solve(np.eye(n) - alpha * S, (1 - alpha) * x0)
    assert np.allclose(oracle.propagate(indptr, indices, x0, alpha, 300, s, s), limit, rtol=1e-10, atol=1e-10)
