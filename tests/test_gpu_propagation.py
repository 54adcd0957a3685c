"""GPU parity of the weighted sum aggregation X <- diag(dst_scale) A diag(src_scale) X (the propagation step of
label-propagation post-processing, Sec. 4.2) with the float64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _hub_graph(n=6000, e=60000, d_max=600.0, seed=9):
    s, d = workloads.chung_lu_edges(workloads.ChungLuSpec(n=n, e=e, gamma=2.1, d_max=d_max, seed=seed))
    return n, s, d


@pytest.mark.parametrize("F,dtype", [(256, "f32"), (256, "bf16"), (64, "f32"), (8, "bf16"), (5, "f32"), (1000, "f32")])
@pytest.mark.parametrize("threshold", [0, 24])
@pytest.mark.parametrize("which", ["both", "src", "dst"])
def test_weighted_sum_forward_transposed_and_partitions(F, dtype, threshold, which):
    from paper_2111_06483_b200 import api, binding as B
    n, src, dst = _hub_graph()
    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV), k=4, threshold=threshold, build_parts=True)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    feat = workloads.normal_tensor((n, F), 7, 1, dtype=tdt)
    indptr, indices = oracle.csr_from_coo(n, n, src.numpy(), dst.numpy())
    t_indptr, t_indices = oracle.csr_transpose(n, n, indptr, indices)
    # symmetric normalisation: in-degree^-1/2 on the destination side, out-degree^-1/2 on the source side
    din, dout = np.diff(indptr).astype(np.float64), np.diff(t_indptr).astype(np.float64)
    s_dst = np.where(din > 0, 1.0 / np.sqrt(np.maximum(din, 1)), 0.0).astype(np.float32)
    s_src = np.where(dout > 0, 1.0 / np.sqrt(np.maximum(dout, 1)), 0.0).astype(np.float32)
    use_src = s_src if which in ("both", "src") else None
    use_dst = s_dst if which in ("both", "dst") else None
    dv = lambda x: None if x is None else torch.from_numpy(x).to(DEV)
    want = oracle.spmm_scaled(indptr, indices, feat.float().numpy(), use_src, use_dst)
    got = api.spmm_scaled(g.whole, feat.to(DEV), dv(use_src), dv(use_dst))
    # float32 accumulation of deg products; the floor follows the longest row as for the plain sum
    max_deg = int(max(din.max(), dout.max()))
    rms = float(np.sqrt(np.mean(want * want)))
    tol = dict(rtol=2e-2, atol=2e-2 * max(rms, 1e-3)) if dtype == "bf16" else dict(rtol=1e-5, atol=2.0 ** -23 * max_deg)
    allclose_report(got.float().cpu().numpy(), want, what="weighted sum", **tol)
    # the backward pass: the transposed partition with the two scale arrays exchanged
    gout = workloads.normal_tensor((n, F), 7, 2, dtype=tdt)
    want_b = oracle.spmm_scaled(t_indptr, t_indices, gout.float().numpy(), use_dst, use_src)
    got_b = api.spmm_scaled(g.whole.transposed(), gout.to(DEV), dv(use_dst), dv(use_src))
    rms_b = float(np.sqrt(np.mean(want_b * want_b)))
    tol_b = dict(rtol=2e-2, atol=2e-2 * max(rms_b, 1e-3)) if dtype == "bf16" else tol
    allclose_report(got_b.float().cpu().numpy(), want_b, what="weighted sum, transposed", **tol_b)
    # K partitions accumulated one after the other
    out = torch.empty((n, F), dtype=tdt, device=DEV)
    fd = feat.to(DEV)
    ssrc = dv(use_src)
    for q, part in enumerate(g.parts):
        flags = (B.SAR_FIRST if q == 0 else 0) | (B.SAR_LAST if q == 3 else 0)
        ws = torch.empty(B.sar_spmm_workspace_bytes(part, F, B._dtype(fd)), dtype=torch.uint8, device=DEV)
        sq = None if ssrc is None else ssrc[g.bounds[q]:g.bounds[q + 1]]
        B.sar_spmm_agg_scaled(part, fd[g.bounds[q]:g.bounds[q + 1]], F, flags, sq, dv(use_dst), out, ws)
    tol_k = dict(rtol=4e-2, atol=4 * 2.0 ** -8 * float(np.abs(want).max())) if dtype == "bf16" else tol
    allclose_report(out.float().cpu().numpy(), want, what="weighted sum K=4", **tol_k)


def test_weighted_sum_rejects_the_mean_flag_and_accepts_no_scales():
    from paper_2111_06483_b200 import api, binding as B
    n, src, dst = _hub_graph(n=500, e=4000, d_max=50.0)
    g = api.Graph.from_coo(n, src.to(DEV), dst.to(DEV))
    x = workloads.normal_tensor((n, 16), 3, 1).to(DEV)
    out = torch.empty_like(x)
    ws = torch.empty(B.sar_spmm_workspace_bytes(g.whole, 16, B._dtype(x)), dtype=torch.uint8, device=DEV)
    with pytest.raises(B.SarError) as ei:
        B.sar_spmm_agg_scaled(g.whole, x, 16, B.SAR_FIRST | B.SAR_LAST | B.SAR_MEAN, None, None, out, ws)
    assert ei.value.code == -1
    # without scales it is the plain sum, bit for bit
    B.sar_spmm_agg_scaled(g.whole, x, 16, B.SAR_FIRST | B.SAR_LAST, None, None, out, ws)
    assert torch.equal(out, api.spmm_sum(g.whole, x))
