"""GPU parity of the relational layer (Appendix A) - per-relation mean aggregation, relation weights, sum over
the relations, and the backward pass that rebuilds the aggregates - and of its helpers (degree factors, basis
decomposition, accumulating projection) with the float64 oracle on the same bf16-rounded inputs, through the
C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from helpers import allclose_report, small_problem

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _bf16(a):
    return torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("n,e", [(3, 2), (257, 2000), (5000, 100000)])
def test_degree_factors(n, e):
    from paper_2111_06483_b200 import binding as B
    p = small_problem(n, e, 1, 4, 17)
    indptr = torch.from_numpy(p["indptr"]).to(DEV)
    deg = np.diff(p["indptr"]).astype(np.float32)
    for power, exact in ((-1.0, True), (-0.5, False), (-0.25, False)):
        out = torch.full((n,), float("nan"), dtype=torch.float32, device=DEV)
        B.sar_degree_scale(indptr, power, out)
        with np.errstate(divide="ignore"):
            want = np.where(deg > 0, deg.astype(np.float64) ** power, 0.0)
        got = out.cpu().numpy()
        if exact:  # one correctly rounded float32 division
            assert np.array_equal(got, np.where(deg > 0, np.float32(1.0) / np.maximum(deg, 1), 0).astype(np.float32))
        allclose_report(got.astype(np.float64), want, 1e-6, 0.0, f"degree^{power}")
    with pytest.raises(B.SarError):
        B.sar_degree_scale(indptr, 0.5, out)


@pytest.mark.parametrize("R,Bn,shape", [(4, 2, (256, 256)), (3, 5, (8, 24)), (1, 1, (7, 3))])
def test_basis_decomposition(R, Bn, shape):
    from paper_2111_06483_b200 import api
    rng = np.random.default_rng(5)
    a = torch.from_numpy(rng.standard_normal((R, Bn)).astype(np.float32)).to(DEV)
    V = torch.from_numpy(rng.standard_normal((Bn,) + shape).astype(np.float32)).to(DEV)
    dW = torch.from_numpy(rng.standard_normal((R,) + shape).astype(np.float32)).to(DEV)
    want = oracle.rgcn_basis(_np(a), _np(V))
    scale = float(np.abs(want).max())
    allclose_report(_np(api.rgcn_basis_weights(a, V, torch.float32)), want, 1e-5, 1e-6 * scale, "W fp32")
    allclose_report(_np(api.rgcn_basis_weights(a, V, torch.bfloat16)), want, 2.0 ** -8, 2.0 ** -9 * scale, "W bf16")
    da, dV = api.rgcn_basis_backward(a, V, dW)
    want_da, want_dV = oracle.rgcn_basis_bwd(_np(a), _np(V), _np(dW))
    size = int(np.prod(shape))
    allclose_report(_np(da), want_da, 1e-5, 1e-6 * size ** 0.5, "da")
    allclose_report(_np(dV), want_dV, 1e-5, 1e-6 * float(np.abs(want_dV).max()), "dV")


@pytest.mark.parametrize("n,d_in,d_out", [(1, 8, 8), (1000, 64, 40), (70001, 256, 256)])
def test_accumulating_projection(n, d_in, d_out):
    from paper_2111_06483_b200 import binding as B
    rng = np.random.default_rng(6)
    h = _bf16(rng.standard_normal((n, d_in))).to(DEV)
    w = _bf16(rng.standard_normal((d_in, d_out)) / d_in ** 0.5).to(DEV)
    z = _bf16(rng.standard_normal((n, d_out))).to(DEV)
    want = _np(z) + oracle.linear(_np(h), _np(w))
    ws = torch.empty(B.sar_linear_workspace_bytes(n, d_in, d_out), dtype=torch.uint8, device=DEV)
    B.sar_linear_accumulate(h, w, z, ws)
    allclose_report(_np(z), want, 2.0 ** -8, 2.0 ** -8, "z += h W")


def _relation_graphs(n, sizes, seed, k):
    from paper_2111_06483_b200 import api
    ps = [small_problem(n, e, 1, 4, seed + 10 * r) for r, e in enumerate(sizes)]
    graphs = [api.Graph.from_coo(n, torch.from_numpy(p["src"]).to(DEV), torch.from_numpy(p["dst"]).to(DEV), k=k,
                                 build_parts=k > 1) for p in ps]
    return [(p["indptr"], p["indices"]) for p in ps], graphs


@pytest.mark.parametrize("n,sizes,d_in,d_out,k", [
    (300, (2500, 900, 40), 16, 24, 1),
    (300, (2500, 900, 40), 16, 24, 3),
    (20000, (150000, 60000, 90000, 30000), 64, 64, 1),
    (20000, (150000, 60000, 90000, 30000), 64, 64, 4),
    (3000, (40000,), 256, 256, 2),
])
def test_relational_layer_forward_and_backward(n, sizes, d_in, d_out, k):
    from paper_2111_06483_b200 import api
    csr, graphs = _relation_graphs(n, sizes, 23, k)
    rng = np.random.default_rng(7)
    R = len(sizes)
    h = _bf16(rng.standard_normal((n, d_in))).to(DEV)
    W = _bf16(rng.standard_normal((R, d_in, d_out)) / d_in ** 0.5).to(DEV)
    gz = _bf16(rng.standard_normal((n, d_out))).to(DEV)
    z, inv = api.rgcn_layer_forward(graphs, h, W)
    want_z = oracle.rgcn_layer(csr, _np(h), [_np(W[r]) for r in range(R)])
    # bf16 storage of each aggregate and of z after every relation: a few roundings of 2^-9 relative to the terms
    rms = float(np.sqrt((want_z ** 2).mean()))
    allclose_report(_np(z), want_z, 2e-2, 2e-2 * rms, "z")
    dh, dW = api.rgcn_layer_backward(graphs, h, W, inv, gz)
    want_dh, want_dW = oracle.rgcn_layer_bwd(csr, _np(h), [_np(W[r]) for r in range(R)], _np(gz))
    allclose_report(_np(dh), want_dh, 2e-2, 2e-2 * float(np.sqrt((want_dh ** 2).mean())), "dh")
    for r in range(R):
        allclose_report(_np(dW[r]), want_dW[r], 2e-2, 2e-2 * float(np.sqrt((want_dW[r] ** 2).mean())), f"dW[{r}]")
    assert float(np.linalg.norm(_np(z) - want_z) / np.linalg.norm(want_z)) < 5e-3
    assert float(np.linalg.norm(_np(dh) - want_dh) / np.linalg.norm(want_dh)) < 5e-3
