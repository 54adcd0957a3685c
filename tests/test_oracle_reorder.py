"""Pins for the oracle's degree order (graph preparation for locality), CPU only: a library sort, the defining
properties, and the invariance the renumbering must leave intact (Eq. 3 does not depend on how nodes are numbered)."""
import numpy as np

import oracle
from helpers import small_problem


def test_degree_order_is_a_lexicographic_sort():
    rng = np.random.default_rng(3)
    n, e = 200, 1500
    src = rng.integers(0, n, e).astype(np.int32)
    dst = (rng.integers(0, n, e) ** 2 // n).astype(np.int32)      # skewed: many ties and a few hubs
    order, rank = oracle.degree_order(n, src, dst)
    deg = np.bincount(src, minlength=n) + np.bincount(dst, minlength=n)
    want = np.lexsort((np.arange(n), -deg))                        # last key is the primary one
    assert np.array_equal(order, want)
    assert np.array_equal(np.sort(order), np.arange(n))            # a permutation
    assert np.array_equal(order[rank], np.arange(n)) and np.array_equal(rank[order], np.arange(n))
    d = deg[order]
    assert np.all(d[:-1] >= d[1:])
    ties = d[:-1] == d[1:]
    assert np.all(order[:-1][ties] < order[1:][ties])


def test_degree_order_of_a_star_and_of_no_edges():
    n = 6
    src = np.array([1, 2, 3, 4, 5], dtype=np.int32)
    dst = np.zeros(5, dtype=np.int32)
    order, rank = oracle.degree_order(n, src, dst)
    assert order.tolist() == [0, 1, 2, 3, 4, 5] and rank.tolist() == [0, 1, 2, 3, 4, 5]
    src = np.array([0, 1, 2, 3, 4], dtype=np.int32)
    dst = np.full(5, 5, dtype=np.int32)                            # the hub is the last node
    order, rank = oracle.degree_order(n, src, dst)
    assert order.tolist() == [5, 0, 1, 2, 3, 4] and rank.tolist() == [1, 2, 3, 4, 5, 0]
    order, rank = oracle.degree_order(4, np.zeros(0, np.int32), np.zeros(0, np.int32))
    assert order.tolist() == [0, 1, 2, 3]


def test_attention_layer_does_not_depend_on_the_numbering():
    p = small_problem(70, 600, 2, 4, 11)
    n = 70
    order, rank = oracle.degree_order(n, p["src"], p["dst"])
    f = oracle.gat_fwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], 0.2)
    b = oracle.gat_bwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], f.alpha, p["gout"], 0.2)
    indptr2, indices2 = oracle.csr_from_coo(n, n, rank[p["src"]], rank[p["dst"]])
    q = {k: p[k][order] for k in ("feat", "el", "er", "gout")}    # node i of the new numbering is node order[i]
    f2 = oracle.gat_fwd(indptr2, indices2, q["feat"], q["el"], q["er"], 0.2)
    b2 = oracle.gat_bwd(indptr2, indices2, q["feat"], q["el"], q["er"], f2.alpha, q["gout"], 0.2)
    assert np.allclose(f2.out[rank], f.out, rtol=1e-12, atol=1e-14)
    assert np.array_equal(f2.m[rank], f.m)
    assert np.allclose(f2.d[rank], f.d, rtol=1e-12)
    assert np.allclose(b2.dfeat[rank], b.dfeat, rtol=1e-10, atol=1e-13)
    assert np.allclose(b2.del_[rank], b.del_, rtol=1e-10, atol=1e-13)
    assert np.allclose(b2.der[rank], b.der, rtol=1e-10, atol=1e-13)
