"""Shared test utilities: small seeded problems and the dense brute-force definitions
that pin the oracle.  Nothing here is used by the CUDA path."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import workloads


def small_problem(n, e, H, F, seed, self_loops=False, dtype="f32", empty_rows=0):
    """Uniform random directed multigraph + N(0,1) node tensors, as numpy arrays.

    `empty_rows` destinations get all their in-edges removed (redirected to node 0)."""
    src, dst = workloads.uniform_edges(n, e, seed, self_loops)
    src, dst = src.numpy().copy(), dst.numpy().copy()
    if empty_rows:
        kill = np.arange(n - empty_rows, n)
        dst[np.isin(dst, kill)] = 0
    t = workloads.make_node_inputs(n, H, F, seed, dtype=dtype)
    arr = {k: v.float().numpy() for k, v in t.items()}
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    return dict(n=n, src=src, dst=dst, indptr=indptr, indices=indices, H=H, F=F, **arr)


def count_matrix(n_dst, n_src, src, dst):
    """C[i,j] = number of edges j -> i."""
    C = np.zeros((n_dst, n_src), dtype=np.float64)
    np.add.at(C, (dst, src), 1.0)
    return C


def dense_gat(C, feat, el, er, slope):
    """Eq. 3 on a dense count matrix, numpy float64: returns (P[i,j,h], out[i,h,f])."""
    feat, el, er = feat.astype(np.float64), el.astype(np.float64), er.astype(np.float64)
    s = el[:, None, :] + er[None, :, :]                     # [i,j,h]
    e = np.where(s > 0, s, slope * s)
    e = np.where(C[:, :, None] > 0, e, -np.inf)
    mx = e.max(axis=1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    w = C[:, :, None] * np.exp(e - mx)
    den = w.sum(axis=1, keepdims=True)
    P = np.divide(w, den, out=np.zeros_like(w), where=den > 0)
    out = np.einsum("ijh,jhf->ihf", P, feat)
    return P, out


def dense_gat_torch(C, feat, el, er, slope):
    """Same dense formulation with torch float64 ops, differentiable in feat, el, er."""
    s = el[:, None, :] + er[None, :, :]
    e = torch.nn.functional.leaky_relu(s, negative_slope=slope)
    mask = (C > 0)[:, :, None]
    e = torch.where(mask, e, torch.full_like(e, -1e300))
    mx = e.max(dim=1, keepdim=True).values.detach()
    w = C[:, :, None] * torch.exp(e - mx)
    den = w.sum(dim=1, keepdim=True)
    P = torch.where(den > 0, w / torch.where(den > 0, den, torch.ones_like(den)), torch.zeros_like(w))
    return torch.einsum("ijh,jhf->ihf", P, feat)


TOLERANCE_USE = []   # (what, worst error, share of the tolerance used) of every check since the last drain


def allclose_report(got, want, rtol, atol, what=""):
    """|got - want| <= atol + rtol * |want| element by element; records the largest error seen and the
    share of its tolerance that it used (drained into the test's properties by conftest.py)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    both_inf = np.isinf(got) & np.isinf(want) & (np.sign(got) == np.sign(want))
    with np.errstate(invalid="ignore"):  # inf - inf where both are the same infinity
        err = np.where(both_inf, 0.0, np.abs(got - want))
    tol = atol + rtol * np.where(both_inf, 0.0, np.abs(want))
    bad = ~(err <= tol)
    if got.size:
        with np.errstate(invalid="ignore", divide="ignore"):
            use = np.where(tol > 0, err / tol, np.where(err > 0, np.inf, 0.0))
        use = np.where(np.isnan(use), np.inf, use)
        TOLERANCE_USE.append((what, float(np.nanmax(np.where(np.isnan(err), np.inf, err))), float(use.max())))
    if bad.any():
        k = np.argmax(np.where(bad, err - tol, -np.inf))
        idx = np.unravel_index(k, got.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside rtol={rtol} atol={atol}; worst at {idx}: "
                             f"got {got[idx]!r} want {want[idx]!r} err {err[idx]:.3e}")
