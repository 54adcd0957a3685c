"""Pins for the oracle's forward functions (CPU only).

Each test fixes the oracle against something that is not the oracle: a dense brute force of
Eq. 3, a scipy.sparse product, scipy's softmax, closed forms, or an algebraic invariant."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.sparse as sp
import scipy.special

import oracle
from helpers import allclose_report, count_matrix, dense_gat, small_problem

GOLD = os.path.join(os.path.dirname(__file__), "golden", "eq3_closed_form.json")


def _fwd(p, slope=0.2, **over):
    a = {**p, **over}
    return oracle.gat_fwd(a["indptr"], a["indices"], a["feat"], a["el"], a["er"], slope)


@pytest.mark.parametrize("n,e,H,F,seed,loops", [(7, 20, 1, 1, 1, False), (40, 300, 3, 5, 2, True),
                                                (64, 900, 4, 8, 3, False)])
def test_forward_matches_dense_masked_softmax(n, e, H, F, seed, loops):
    p = small_problem(n, e, H, F, seed, self_loops=loops, empty_rows=3)
    C = count_matrix(n, n, p["src"], p["dst"])
    P, out = dense_gat(C, p["feat"], p["el"], p["er"], 0.2)
    r = _fwd(p)
    allclose_report(r.out, out, 1e-12, 1e-13, "out vs dense")
    # per-edge alpha * multiplicity == dense P entry
    dst_of_edge = np.repeat(np.arange(n), np.diff(p["indptr"]))
    got = np.zeros_like(P)
    np.add.at(got, (dst_of_edge, p["indices"]), r.alpha)
    allclose_report(got, P, 1e-12, 1e-14, "alpha vs dense")
    # direction matters: swapping el/er roles must NOT reproduce the result on a directed graph
    _, out_swapped = dense_gat(C, p["feat"], p["er"], p["el"], 0.2)
    assert np.abs(out_swapped - out).max() > 1e-3


def test_forward_golden_closed_form():
    g = json.load(open(GOLD))
    ln2 = np.log(2.0)
    n = g["n"]
    indptr, indices = oracle.csr_from_coo(n, n, g["src"], g["dst"])
    el = (np.array(g["el_over_ln2"]) * ln2).astype(np.float32).reshape(n, 1)
    er = (np.array(g["er_over_ln2"]) * ln2).astype(np.float32).reshape(n, 1)
    feat = np.array(g["feat"], dtype=np.float32).reshape(n, 1, 1)
    r = oracle.gat_fwd(indptr, indices, feat, el, er, g["slope"])
    want_alpha = np.array([float(Fraction(x)) for x in g["expect"]["alpha"]]).reshape(-1, 1)
    allclose_report(r.alpha, want_alpha, 1e-6, 0, "alpha")      # inputs are float32-rounded logs
    assert abs(r.out[0, 0, 0] - float(Fraction(g["expect"]["out0"]))) < 1e-5
    assert abs(r.m[0, 0] - g["expect"]["m0_over_ln2"] * ln2) < 1e-6
    assert abs(r.d[0, 0] - float(Fraction(g["expect"]["d0"]))) < 1e-6
    assert np.all(r.out[1:] == 0) and np.all(r.d[1:] == 0) and np.all(np.isneginf(r.m[1:]))


def test_softmax_weights_sum_to_one_and_constant_features():
    p = small_problem(300, 3000, 4, 8, 5, empty_rows=10)
    r = _fwd(p)
    deg = np.diff(p["indptr"])
    dst_of_edge = np.repeat(np.arange(p["n"]), deg)
    s = np.zeros((p["n"], p["H"]))
    np.add.at(s, dst_of_edge, r.alpha)
    allclose_report(s[deg > 0], np.ones_like(s[deg > 0]), 1e-13, 0, "sum alpha")
    assert np.all(s[deg == 0] == 0)
    ones = np.ones_like(p["feat"])
    r1 = _fwd(p, feat=ones)
    allclose_report(r1.out[deg > 0], np.ones_like(r1.out[deg > 0]), 1e-13, 0, "feat==1")
    assert np.all(r1.out[deg == 0] == 0)


def test_zero_scores_give_neighbour_mean_scipy():
    p = small_problem(500, 6000, 2, 6, 6, empty_rows=5)
    z = np.zeros_like(p["el"])
    r = _fwd(p, el=z, er=z)
    n = p["n"]
    A = sp.csr_matrix((np.ones(len(p["indices"])), p["indices"], p["indptr"]), shape=(n, n))
    deg = np.asarray(A.sum(axis=1)).ravel()
    mean = A @ p["feat"].reshape(n, -1).astype(np.float64)
    mean[deg > 0] /= deg[deg > 0, None]
    allclose_report(r.out.reshape(n, -1), mean, 1e-12, 1e-14, "mean")
    # and the sum-aggregation oracle against the same scipy product (Eq. 2)
    f2 = p["feat"].reshape(n, -1)
    allclose_report(oracle.spmm(p["indptr"], p["indices"], f2), A @ f2.astype(np.float64), 1e-12, 1e-14, "spmm")
    allclose_report(oracle.spmm(p["indptr"], p["indices"], f2, mean=True), mean, 1e-12, 1e-14, "spmm mean")
    # backward of the sum = the same routine on the transposed graph
    t_indptr, t_indices = oracle.csr_transpose(n, n, p["indptr"], p["indices"])
    g2 = p["gout"].reshape(n, -1)
    allclose_report(oracle.spmm(t_indptr, t_indices, g2), A.T @ g2.astype(np.float64), 1e-12, 1e-14, "spmm bwd")


def test_single_in_edge_copies_the_source_row():
    n = 50
    src = (np.arange(n) * 7 + 3) % n
    dst = np.arange(n)
    p = small_problem(n, 10, 3, 4, 7)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    r = oracle.gat_fwd(indptr, indices, p["feat"], p["el"], p["er"], 0.2)
    assert np.array_equal(r.out, p["feat"][src].astype(np.float64))
    assert np.all(r.d == 1.0)


def test_slope_one_makes_destination_term_irrelevant_and_shift_invariance():
    p = small_problem(200, 2500, 4, 4, 8)
    a = _fwd(p, slope=1.0)
    b = _fwd(p, slope=1.0, el=p["el"] * -3.0 + 1.0)
    allclose_report(a.out, b.out, 1e-6, 1e-7, "slope=1")          # float32 el => tiny input rounding
    # moving a constant from er to el changes no score (power-of-two shift keeps float32 sums exact)
    c = _fwd(p, el=(p["el"] + 0.5).astype(np.float32), er=(p["er"] - 0.5).astype(np.float32))
    allclose_report(c.out, _fwd(p).out, 1e-6, 1e-7, "shift")


def test_large_logits_are_stable_and_match_scipy_softmax():
    p = small_problem(120, 1500, 2, 3, 9)
    el, er = p["el"] * 1e3, p["er"] * 1e3
    r = _fwd(p, el=el, er=er)
    assert np.isfinite(r.out).all()
    for i in range(p["n"]):
        lo, hi = p["indptr"][i], p["indptr"][i + 1]
        if lo == hi:
            continue
        s = el[i].astype(np.float64)[None, :] + er[p["indices"][lo:hi]].astype(np.float64)
        e = np.where(s > 0, s, 0.2 * s)
        allclose_report(r.alpha[lo:hi], scipy.special.softmax(e, axis=0), 1e-12, 1e-300, f"row {i}")
        lse = scipy.special.logsumexp(e, axis=0)
        allclose_report(r.m[i] + np.log(r.d[i]), lse, 1e-12, 0, "m + log d == logsumexp")
    # a naive exp(e) would overflow here
    with np.errstate(over="ignore"):
        assert np.isinf(np.exp(r.e.max()))


@pytest.mark.parametrize("k", [1, 2, 3, 7, 8, 16, 150])
def test_sequential_merge_equals_definition(k):
    p = small_problem(150, 2200, 3, 5, 10, empty_rows=4)
    ref = _fwd(p)
    bounds = oracle.partition_bounds(p["n"], k)
    split = oracle.csr_split(p["n"], p["indptr"], p["indices"], bounds)
    out, m, d = oracle.gat_fwd_seq(split, p["feat"], p["el"], p["er"], 0.2)
    assert np.array_equal(m, ref.m)                                  # the running max ends exact
    allclose_report(out, ref.out, 1e-13, 1e-15, "seq out")
    allclose_report(d, ref.d, 1e-13, 0, "seq d")
    rng = np.random.default_rng(k)
    out2, m2, d2 = oracle.gat_fwd_seq(split, p["feat"], p["el"], p["er"], 0.2, order=rng.permutation(k))
    assert np.array_equal(m2, ref.m)
    allclose_report(out2, ref.out, 1e-13, 1e-15, "permuted order")
    allclose_report(d2, ref.d, 1e-13, 0, "permuted d")


def test_sequential_merge_with_huge_logits():
    p = small_problem(80, 900, 2, 3, 11)
    el, er = p["el"] * 500.0, p["er"] * 500.0
    ref = oracle.gat_fwd(p["indptr"], p["indices"], p["feat"], el, er, 0.2)
    split = oracle.csr_split(p["n"], p["indptr"], p["indices"], oracle.partition_bounds(p["n"], 5))
    out, m, d = oracle.gat_fwd_seq(split, p["feat"], el, er, 0.2)
    assert np.isfinite(out).all() and np.array_equal(m, ref.m)
    allclose_report(out, ref.out, 1e-12, 1e-15, "seq huge")
