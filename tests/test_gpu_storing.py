"""The non-rematerialising baseline (sar_gat_fwd_storing / sar_gat_bwd_storing): the attention coefficients it
writes are compared with the oracle's per-edge alpha element by element, its outputs and gradients with the
oracle's, and the memory it needs is checked to grow with the edge count where the rematerialising path's does
not."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2111_06483_b200 import api, binding as B

DEV = "cuda"


def _run(cfg, dtype):
    src, dst = workloads.make_graph(cfg)
    n, H, F = cfg.n, cfg.heads, cfg.feat
    host = workloads.make_node_inputs(n, H, F, cfg.seed, dtype=dtype)
    t = {k: v.to(DEV) for k, v in host.items()}
    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV), k=1)
    nnz = g.nnz
    alpha = torch.full((nnz, H), float("nan"), device=DEV)
    out = torch.empty_like(t["feat"])
    B.sar_gat_fwd_storing(g.whole, t["feat"], t["el"], t["er"], H, F, cfg.slope, alpha, out)
    dfeat = torch.empty_like(t["feat"])
    del_, der = torch.empty((n, H), device=DEV), torch.empty((n, H), device=DEV)
    ws = torch.empty(B.sar_gat_storing_workspace_bytes(g.whole, H), dtype=torch.uint8, device=DEV)
    B.sar_gat_bwd_storing(g.whole, t["feat"], t["el"], t["er"], alpha, t["gout"], H, F, cfg.slope, dfeat, del_, der, ws)
    torch.cuda.synchronize()
    h = {k: v.float().numpy() for k, v in host.items()}
    indptr, indices = oracle.csr_from_coo(n, n, src.numpy(), dst.numpy())
    assert np.array_equal(g.whole.indices.cpu().numpy(), indices)      # alpha's row order is the CSR's edge order
    f = oracle.gat_fwd(indptr, indices, h["feat"], h["el"], h["er"], cfg.slope)
    b = oracle.gat_bwd(indptr, indices, h["feat"], h["el"], h["er"], f.alpha, h["gout"], cfg.slope)
    max_out_deg = int((g.whole.t_indptr[1:] - g.whole.t_indptr[:-1]).max())
    return (alpha, out, dfeat, del_, der), (f, b), max_out_deg


@pytest.mark.parametrize("name,scale,dtype", [("tiny", None, "f32"), ("seqpart", None, "f32"), ("seqpart", 0.3, "bf16")])
def test_stored_attention_matches_the_oracles_alpha(name, scale, dtype):
    cfg = workloads.CONFIGS[name]
    if scale:
        cfg = cfg.scaled(scale)
    (alpha, out, dfeat, del_, der), (f, b), max_out_deg = _run(cfg, dtype)
    # The baseline adds a row's terms one after the other in float32 (no pairwise or lane-parallel sums): a source
    # with d out-edges carries up to 2^-24 * d * |term| of rounding, so the gradient floor follows the longest row.
    floor = max(1e-5, 2.0 ** -23 * max_out_deg)
    allclose_report(alpha.cpu().numpy(), f.alpha, 1e-5, 1e-7, "alpha")          # element by element, every edge and head
    rms = lambda x: max(float(np.sqrt(np.mean(np.square(x)))), 1.0)
    if dtype == "bf16":
        allclose_report(out.float().cpu().numpy(), f.out, 2e-2, 4 * 2.0 ** -9 * rms(f.out), "out")
        allclose_report(dfeat.float().cpu().numpy(), b.dfeat, 2e-2, 4 * 2.0 ** -9 * rms(b.dfeat), "dfeat")
    else:
        allclose_report(out.cpu().numpy(), f.out, 1e-5, 1e-6, "out")
        allclose_report(dfeat.cpu().numpy(), b.dfeat, 1e-4, floor * rms(b.dfeat), "dfeat")
    allclose_report(del_.cpu().numpy(), b.del_, 1e-4, 1e-5 * rms(b.del_), "del")
    allclose_report(der.cpu().numpy(), b.der, 1e-4, floor * rms(b.der), "der")


def test_storing_needs_memory_in_proportion_to_the_edges():
    cfg = workloads.CONFIGS["seqpart"]
    src, dst = workloads.make_graph(cfg, device=DEV)
    g = api.Graph.from_coo(cfg.n, src, dst, k=1)
    kept = 4 * g.nnz * cfg.heads                                   # alpha, kept from the forward to the backward pass
    assert B.sar_gat_storing_workspace_bytes(g.whole, cfg.heads) >= 4 * g.nnz * cfg.heads + 4 * g.nnz
    assert kept > 3 * (2 * 4 * cfg.n * cfg.heads)                  # against the 8 bytes per (node, head) of (m, d)
