"""Pins for the oracle's backward function (CPU only): finite differences, torch autograd on a
dense formulation of Eq. 3, a hand-computed fixture, and invariants of the softmax Jacobian."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report, count_matrix, dense_gat_torch, small_problem

GOLD = os.path.join(os.path.dirname(__file__), "golden", "eq3_closed_form.json")


def _fwd_bwd(p, slope=0.2):
    f = oracle.gat_fwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], slope)
    b = oracle.gat_bwd(p["indptr"], p["indices"], p["feat"], p["el"], p["er"], f.alpha, p["gout"], slope)
    return f, b


def _loss(p, feat, el, er, slope):
    """<gout, out> with float64 inputs evaluated through a dense numpy formulation-free path:
    the oracle itself only accepts float32 storage, so finite differences use this local
    float64 edge loop (independent code)."""
    n, H, F = p["n"], p["H"], p["F"]
    total = 0.0
    for i in range(n):
        lo, hi = p["indptr"][i], p["indptr"][i + 1]
        if lo == hi:
            continue
        js = p["indices"][lo:hi]
        s = el[i][None, :] + er[js]
        e = np.where(s > 0, s, slope * s)
        w = np.exp(e - e.max(axis=0, keepdims=True))
        a = w / w.sum(axis=0, keepdims=True)
        out = np.einsum("th,thf->hf", a, feat[js])
        total += float((out * p["gout"][i]).sum())
    return total


def test_backward_matches_central_finite_differences():
    p = small_problem(12, 40, 2, 3, 21, empty_rows=1)
    _, b = _fwd_bwd(p)
    feat, el, er = (p[k].astype(np.float64) for k in ("feat", "el", "er"))
    h = 1e-6
    for name, base, grad in (("feat", feat, b.dfeat), ("el", el, b.del_), ("er", er, b.der)):
        num = np.zeros_like(base)
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            args = dict(feat=feat, el=el, er=er)
            plus, minus = base.copy(), base.copy()
            plus[idx] += h
            minus[idx] -= h
            num[idx] = (_loss(p, **{**args, name: plus}, slope=0.2) -
                        _loss(p, **{**args, name: minus}, slope=0.2)) / (2 * h)
        allclose_report(grad, num, 1e-6, 1e-8, f"d{name} vs finite differences")


@pytest.mark.parametrize("n,e,H,F,seed", [(30, 200, 2, 4, 22), (60, 800, 4, 8, 23)])
def test_backward_matches_torch_autograd_on_dense_formulation(n, e, H, F, seed):
    p = small_problem(n, e, H, F, seed, self_loops=True, empty_rows=2)
    _, b = _fwd_bwd(p)
    C = torch.from_numpy(count_matrix(n, n, p["src"], p["dst"]))
    feat = torch.tensor(p["feat"], dtype=torch.float64, requires_grad=True)
    el = torch.tensor(p["el"], dtype=torch.float64, requires_grad=True)
    er = torch.tensor(p["er"], dtype=torch.float64, requires_grad=True)
    out = dense_gat_torch(C, feat, el, er, 0.2)
    (out * torch.tensor(p["gout"], dtype=torch.float64)).sum().backward()
    allclose_report(b.dfeat, feat.grad.numpy(), 1e-11, 1e-13, "dfeat vs autograd")
    allclose_report(b.del_, el.grad.numpy(), 1e-10, 1e-12, "del vs autograd")
    allclose_report(b.der, er.grad.numpy(), 1e-10, 1e-12, "der vs autograd")


def test_backward_golden_closed_form():
    g = json.load(open(GOLD))
    ln2 = np.log(2.0)
    n = g["n"]
    indptr, indices = oracle.csr_from_coo(n, n, g["src"], g["dst"])
    el = (np.array(g["el_over_ln2"]) * ln2).astype(np.float32).reshape(n, 1)
    er = (np.array(g["er_over_ln2"]) * ln2).astype(np.float32).reshape(n, 1)
    feat = np.array(g["feat"], dtype=np.float32).reshape(n, 1, 1)
    gout = np.array(g["gout"], dtype=np.float32).reshape(n, 1, 1)
    f = oracle.gat_fwd(indptr, indices, feat, el, er, g["slope"])
    b = oracle.gat_bwd(indptr, indices, feat, el, er, f.alpha, gout, g["slope"])
    ex = g["expect"]
    fr = lambda xs: np.array([float(Fraction(x)) for x in xs])
    assert abs(b.D[0, 0] - float(Fraction(ex["D0"]))) < 1e-5
    assert abs(b.del_[0, 0] - float(Fraction(ex["del0"]))) < 1e-5
    allclose_report(b.der.ravel(), fr(ex["der"]), 0, 1e-5, "der")
    allclose_report(b.dfeat.ravel(), fr(ex["dfeat"]), 0, 1e-6, "dfeat")


def test_backward_invariants():
    p = small_problem(400, 5000, 4, 8, 24, empty_rows=6)
    f, b = _fwd_bwd(p)
    deg = np.diff(p["indptr"])
    gout = p["gout"].astype(np.float64)
    # D is the row dot <gout, out>
    allclose_report(b.D, (gout * f.out).sum(axis=2), 1e-11, 1e-13, "D == <gout,out>")
    # every edge hands alpha*gout to its source and alpha sums to one per destination
    allclose_report(b.dfeat.sum(axis=0), gout[deg > 0].sum(axis=0), 1e-11, 1e-12, "sum dfeat")
    # del and der are two groupings of the same per-edge ds
    allclose_report(b.del_.sum(axis=0), b.der.sum(axis=0), 1e-10, 1e-12, "sum del == sum der")
    assert np.all(b.del_[deg == 0] == 0)
    # slope = 1: LeakyReLU is the identity and the softmax Jacobian's rows sum to zero
    f1, b1 = _fwd_bwd(p, slope=1.0)
    assert np.abs(b1.del_).max() < 1e-12


def test_leaky_relu_derivative_at_zero_is_the_slope():
    """The paper does not say what the derivative at 0 is; both sides take `slope`.
    Destination 0 has in-edges from 1 (score exactly 0) and 2 (score ln 2): alpha = 1/3, 2/3;
    with feat = (3, 0) and gout = 1: dalpha = (3, 0), D = 1, de = (2/3, -2/3), ds = (slope*2/3, -2/3)."""
    n = 3
    indptr, indices = oracle.csr_from_coo(n, n, [1, 2], [0, 0])
    el = np.zeros((n, 1), np.float32)
    er = np.array([0, 0, np.log(2.0)], np.float32).reshape(n, 1)
    feat = np.array([0, 3, 0], np.float32).reshape(n, 1, 1)
    gout = np.array([1, 0, 0], np.float32).reshape(n, 1, 1)
    f = oracle.gat_fwd(indptr, indices, feat, el, er, 0.2)
    b = oracle.gat_bwd(indptr, indices, feat, el, er, f.alpha, gout, 0.2)
    allclose_report(b.der.ravel(), [0.0, 0.2 * 2 / 3, -2 / 3], 1e-6, 1e-9, "der at s=0")
    assert abs(b.del_[0, 0] - (0.2 * 2 / 3 - 2 / 3)) < 1e-6
