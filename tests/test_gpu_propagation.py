"""GPU parity of the weighted sum aggregation X <- diag(dst_scale) A diag(src_scale) X (the propagation step of
label-propagation post-processing, Sec. 4.2) with the float64 oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report, small_problem

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
    # float32 accumulation of deg products, eight slots at a time and then the groups of eight; the floor follows the
    # longest chain of additions as for the plain sum.  A bf16 output is rounded once (2^-9 relative).
    max_deg = int(max(din.max(), dout.max()))
    rms = float(np.sqrt(np.mean(want * want)))
    tol = (dict(rtol=2.0 ** -7, atol=2.0 ** -9 * max(rms, 1e-3)) if dtype == "bf16"
           else dict(rtol=1e-5, atol=2.0 ** -23 * (8 + max_deg / 8)))
    allclose_report(got.float().cpu().numpy(), want, what="weighted sum", **tol)
    # the backward pass: the transposed partition with the two scale arrays exchanged
    gout = workloads.normal_tensor((n, F), 7, 2, dtype=tdt)
    want_b = oracle.spmm_scaled(t_indptr, t_indices, gout.float().numpy(), use_dst, use_src)
    got_b = api.spmm_scaled(g.whole.transposed(), gout.to(DEV), dv(use_dst), dv(use_src))
    rms_b = float(np.sqrt(np.mean(want_b * want_b)))
    tol_b = dict(rtol=2.0 ** -7, atol=2.0 ** -9 * max(rms_b, 1e-3)) if dtype == "bf16" else tol
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
    tol_k = dict(rtol=4 * 2.0 ** -8, atol=4 * 2.0 ** -9 * float(np.abs(want).max())) if dtype == "bf16" else tol
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


@pytest.mark.parametrize("n,dtype", [(1, "f32"), (1000, "f32"), (4099, "bf16"), (1 << 20, "bf16"), ((1 << 20) + 3, "f32")])
def test_axpby(n, dtype):
    from paper_2111_06483_b200 import binding as B
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    rng = np.random.default_rng(n)
    x = torch.from_numpy(rng.standard_normal(n).astype(np.float32)).to(tdt).to(DEV)
    y = torch.from_numpy(rng.standard_normal(n).astype(np.float32)).to(tdt).to(DEV)
    want = 0.25 * x.double().cpu().numpy() - 1.5 * y.double().cpu().numpy()
    B.sar_axpby(0.25, x, -1.5, y)
    tol = dict(rtol=1e-6, atol=1e-6) if dtype == "f32" else dict(rtol=2.0 ** -8, atol=2.0 ** -8)
    allclose_report(y.double().cpu().numpy(), want, what="a x + b y", **tol)
    # an unaligned view takes the element-wise path
    if n > 8:
        xs, ys = x[1:], y[1:]
        want = 2.0 * xs.double().cpu().numpy() + 0.5 * ys.double().cpu().numpy()
        B.sar_axpby(2.0, xs, 0.5, ys)
        allclose_report(ys.double().cpu().numpy(), want, what="a x + b y, unaligned", **tol)
    with pytest.raises(B.SarError):
        B.sar_axpby(1.0, y, 1.0, y)


@pytest.mark.parametrize("dtype,k", [("f32", 1), ("f32", 3), ("bf16", 1), ("bf16", 4)])
def test_iterated_propagation(dtype, k):
    from paper_2111_06483_b200 import api
    n, e, F, alpha, iters = 3000, 20000, 24, 0.8, 6
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    p = small_problem(n, e, 1, 4, 77)
    src = np.concatenate([p["src"], p["dst"]]).astype(np.int32)   # undirected: every edge in both directions
    dst = np.concatenate([p["dst"], p["src"]]).astype(np.int32)
    indptr, indices = oracle.csr_from_coo(n, n, src, dst)
    g = api.Graph.from_coo(n, torch.from_numpy(src).to(DEV), torch.from_numpy(dst).to(DEV), k=k, build_parts=k > 1)
    s_src, s_dst = api.sym_norm_scales(g)
    deg = np.diff(indptr).astype(np.float64)
    want_scale = np.where(deg > 0, 1.0 / np.sqrt(np.maximum(deg, 1)), 0.0)
    allclose_report(s_dst.cpu().numpy().astype(np.float64), want_scale, 1e-6, 0.0, "in-degree^-1/2")
    allclose_report(s_src.cpu().numpy().astype(np.float64), want_scale, 1e-6, 0.0, "out-degree^-1/2")
    x0 = torch.from_numpy(np.random.default_rng(4).standard_normal((n, F)).astype(np.float32)).to(tdt)
    got = api.propagate(g, x0.to(DEV), alpha, iters, s_src, s_dst)
    want = oracle.propagate(indptr, indices, x0.float().numpy(), alpha, iters,
                            s_src.cpu().numpy(), s_dst.cpu().numpy())
    tol = dict(rtol=1e-5, atol=1e-5) if dtype == "f32" else dict(rtol=2e-2, atol=2e-2)  # bf16: two roundings per step
    allclose_report(got.float().cpu().numpy(), want, what=f"{iters} propagation steps", **tol)
