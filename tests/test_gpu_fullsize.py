"""GPU parity at the full sizes of the named workloads, in the launch configurations bench.py times
(the fused calls over the un-split graph and the call-by-call sequence over the K partitions, long-row
plans with the default threshold).

The oracle cannot run 300 M edges in test time, so outputs are SAMPLED: a sub-problem that contains
every edge the sampled outputs depend on is cut out with torch indexing, handed to the oracle, and
compared element by element; invariants that hold at any size cover the rest.
  forward / del : sampled destinations with ALL their in-edges (out, m, d, del depend on nothing else)
  dfeat / der   : sampled sources with all their out-edges, plus, for every destination those edges
                  reach, ALL of its in-edges (so that the softmax statistics of the sub-problem are exact)
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from helpers import allclose_report

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2111_06483_b200 import api

DEV = "cuda"


def _rows_subgraph(indptr, indices, rows):
    """CSR restricted to `rows` (device tensors): returns (sub_indptr[len(rows)+1], cols) on the device."""
    deg = indptr[rows + 1] - indptr[rows]
    sub_indptr = torch.zeros(rows.numel() + 1, dtype=torch.int64, device=rows.device)
    sub_indptr[1:] = torch.cumsum(deg, 0)
    total = int(sub_indptr[-1])
    owner = torch.repeat_interleave(torch.arange(rows.numel(), device=rows.device), deg)
    pos = torch.arange(total, device=rows.device) - sub_indptr[owner] + indptr[rows][owner]
    return sub_indptr, indices[pos].long()


def _tol(dtype, want, grad=False, stored=True):
    """The tolerances of test_gpu_parity.py: float32 outputs 1e-5 / 1e-6, float32 gradients 1e-4 with a floor of
    1e-5 x max(RMS, 1); arrays stored in bf16 (out, dfeat) 2^-7 relative plus 2^-9 of the RMS; del and der are
    float32 arrays in every variant."""
    x = np.asarray(want, dtype=np.float64)
    scale = max(float(np.sqrt(np.mean(x * x))) if x.size else 0.0, 1.0)
    if dtype == "bf16" and stored:
        return dict(rtol=2.0 ** -7, atol=2.0 ** -9 * scale)
    return dict(rtol=1e-4, atol=1e-5 * scale) if grad else dict(rtol=1e-5, atol=1e-6)


def _run_schedule(g, t, cfg, dtype, mode):
    """Forward + backward of one layer in one schedule of the K partitions; returns the six outputs."""
    feat, gout, el, er = t["feat"], t["gout"], t["el"], t["er"]
    if mode == "fused":
        out, m, d = api.gat_forward(g, feat, el, er, cfg.slope)
        dfeat, del_, der = api.gat_backward(g, feat, el, er, m, d, gout, cfg.slope)
    else:
        # K calls of sar_gat_fwd with the running state in device memory (Algorithm 1), then
        # sar_gat_bwd_prepare and K calls of sar_gat_bwd (Algorithm 2).  With bf16 storage the row dot is
        # formed from the float32 numerator the last forward call leaves behind.
        keep = dtype == "bf16" and g.k > 1
        fw = api.gat_forward(g, feat, el, er, cfg.slope, mode="stateful", keep_numerator=keep)
        out, m, d = fw[:3]
        dfeat, del_, der = api.gat_backward(g, feat, el, er, m, d, gout, cfg.slope, out=out, mode="stateful",
                                            acc=fw[3] if keep else None)
        del fw
    torch.cuda.synchronize()
    return out, m, d, dfeat, del_, der


@pytest.mark.parametrize("name,dtype", [("seqpart", "f32"), ("medium", "f32"), ("medium", "bf16"), ("dense", "bf16"),
                                        ("large", "bf16")])
def test_sampled_rows_at_full_size(name, dtype):
    """Every named workload at its full size, in BOTH schedules of its K partitions: the fused row-stationary
    calls bench.py times by default, and the call-by-call sequence of Algorithm 1 / Algorithm 2 with K
    partitions (seqpart K = 8, medium K = 4, dense K = 8, large K = 16), each against the oracle on sampled
    rows; the running max must end bit-identical in the two schedules."""
    cfg = workloads.CONFIGS[name]
    n, H, F = cfg.n, cfg.heads, cfg.feat
    need = (5 * n * H * F * (2 if dtype == "bf16" else 4) + 4 * n * H * F + 40 * cfg.e) * 1.5
    if torch.cuda.get_device_properties(0).total_memory < need:
        pytest.skip("not enough device memory for this workload")
    src, dst = workloads.make_graph(cfg, device=DEV)
    g = api.Graph.from_coo(n, src, dst, k=cfg.k, build_parts=True)
    del src, dst
    assert g.k == cfg.k and len(g.parts) == cfg.k
    t = workloads.make_node_inputs(n, H, F, cfg.seed, dtype=dtype, device=DEV)
    feat, gout, el, er = t["feat"], t["gout"], t["el"], t["er"]
    W = g.whole
    in_deg = W.indptr[1:] - W.indptr[:-1]
    out_deg = W.t_indptr[1:] - W.t_indptr[:-1]
    empty = in_deg == 0

    # ---- the oracle on two sampled sub-problems ------------------------------------------------------
    gen = torch.Generator(device="cpu").manual_seed(cfg.seed + 100)
    rows = torch.randperm(n, generator=gen)[:3000].to(DEV)
    hubs = torch.topk(in_deg, 3).indices                          # the longest rows go through the segment path
    rows = torch.unique(torch.cat([rows, hubs]))
    sub_indptr, cols = _rows_subgraph(W.indptr, W.indices, rows)
    ucols, inv = torch.unique(cols, return_inverse=True)
    f_sub = feat[ucols].float().cpu().numpy()
    fwd1 = oracle.gat_fwd(sub_indptr.cpu().numpy(), inv.cpu().numpy().astype(np.int32), f_sub,
                          el[rows].cpu().numpy(), er[ucols].cpu().numpy(), cfg.slope)
    bwd1 = oracle.gat_bwd(sub_indptr.cpu().numpy(), inv.cpu().numpy().astype(np.int32), f_sub,
                          el[rows].cpu().numpy(), er[ucols].cpu().numpy(), fwd1.alpha,
                          gout[rows].float().cpu().numpy(), cfg.slope)
    # sampled sources with all their out-edges, plus every in-edge of the destinations those reach
    avg_deg = cfg.e / n
    srcs = torch.randperm(n, generator=gen)[:max(3, int(2000 / avg_deg))].to(DEV)
    if avg_deg < 50:                                             # and a couple of busy sources
        mid = torch.nonzero((out_deg > 200) & (out_deg < 3000)).flatten()[:2]
        srcs = torch.cat([srcs, mid])
    srcs = torch.unique(srcs)
    _, reached = _rows_subgraph(W.t_indptr, W.t_indices, srcs)
    drows = torch.unique(reached)
    sub_indptr, cols = _rows_subgraph(W.indptr, W.indices, drows)
    assert sub_indptr[-1] < 40_000_000, "sample grew too large for the oracle"
    ucols, inv = torch.unique(cols, return_inverse=True)
    f_sub = feat[ucols].float().cpu().numpy()
    ip, ix = sub_indptr.cpu().numpy(), inv.cpu().numpy().astype(np.int32)
    fwd2 = oracle.gat_fwd(ip, ix, f_sub, el[drows].cpu().numpy(), er[ucols].cpu().numpy(), cfg.slope)
    bwd2 = oracle.gat_bwd(ip, ix, f_sub, el[drows].cpu().numpy(), er[ucols].cpu().numpy(), fwd2.alpha,
                          gout[drows].float().cpu().numpy(), cfg.slope)
    where = torch.searchsorted(ucols, srcs)                      # sampled sources inside the sub-problem
    has_out = out_deg[srcs] > 0
    where_np, srcs_ok = where[has_out].cpu().numpy(), srcs[has_out]
    no_out = srcs[~has_out]
    del f_sub, fwd2, cols, inv, ucols

    m_by_mode = {}
    for mode in ("fused", "stateful"):
        out, m, d, dfeat, del_, der = _run_schedule(g, t, cfg, dtype, mode)
        m_by_mode[mode] = m
        # ---- invariants over the whole arrays --------------------------------------------------------
        assert torch.isfinite(out.float()).all() and torch.isfinite(dfeat.float()).all()
        assert (d[empty] == 0).all() and torch.isneginf(m[empty]).all() and (out[empty] == 0).all()
        assert (d[~empty] >= 1.0 - 1e-5).all()                      # the max term contributes exp(0) = 1
        s_del, s_der = del_.double().sum(0), der.double().sum(0)      # two groupings of the same per-edge terms
        scale = float(del_.double().abs().sum(0).max())
        assert float((s_del - s_der).abs().max()) <= (2e-2 if dtype == "bf16" else 1e-4) * max(scale, 1.0) ** 0.5 * 50
        want_sum = gout[~empty].double().sum(0)                       # every edge hands alpha*gout to its source
        got_sum = dfeat.double().sum(0)
        tol = (2e-2 if dtype == "bf16" else 1e-4) * float(gout.double().abs().sum(0).max()) ** 0.5 * 50
        assert float((got_sum - want_sum).abs().max()) <= tol
        # ---- sampled destinations: out, m, d, del ----------------------------------------------------
        allclose_report(out[rows].float().cpu().numpy(), fwd1.out, what=f"out[{mode}]", **_tol(dtype, fwd1.out))
        allclose_report(m[rows].cpu().numpy(), fwd1.m, 1e-6, 1e-6, f"m[{mode}]")
        allclose_report(d[rows].cpu().numpy(), fwd1.d, 1e-5, 1e-6, f"d[{mode}]")
        allclose_report(del_[rows].cpu().numpy(), bwd1.del_, what=f"del[{mode}]", **_tol(dtype, bwd1.del_, grad=True, stored=False))
        # ---- sampled sources: dfeat, der -------------------------------------------------------------
        allclose_report(dfeat[srcs_ok].float().cpu().numpy(), bwd2.dfeat[where_np], what=f"dfeat[{mode}]",
                        **_tol(dtype, bwd2.dfeat[where_np], grad=True))
        allclose_report(der[srcs_ok].cpu().numpy(), bwd2.der[where_np], what=f"der[{mode}]",
                        **_tol(dtype, bwd2.der[where_np], grad=True, stored=False))
        assert (dfeat[no_out] == 0).all() and (der[no_out] == 0).all()
        del out, d, dfeat, del_, der
        torch.cuda.empty_cache()
    assert torch.equal(m_by_mode["fused"], m_by_mode["stateful"])   # the running max is exact in any schedule


def test_stack_host_entry_point_matches_device_calls():
    """sar_gat_stack_host (host buffers in, host buffers out) == the same layers run call by call."""
    from paper_2111_06483_b200 import binding as B
    cfg = workloads.CONFIGS["seqpart"].scaled(0.1)
    n, H, F, L = cfg.n, cfg.heads, cfg.feat, 3
    src, dst = workloads.make_graph(cfg, device=DEV)
    g = api.Graph.from_coo(n, src, dst, k=cfg.k)
    for dtype in ("f32", "bf16"):
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        feat0 = workloads.normal_tensor((n, H, F), 5, 10, dtype=tdt)
        gout = workloads.normal_tensor((n, H, F), 5, 11, dtype=tdt)
        els = [workloads.normal_tensor((n, H), 5, 16 * l + 12) for l in range(L)]
        ers = [workloads.normal_tensor((n, H), 5, 16 * l + 13) for l in range(L)]
        pin = lambda x: x.pin_memory()
        h_out, h_dfeat = pin(torch.empty_like(feat0)), pin(torch.empty_like(feat0))
        h_del = [pin(torch.empty((n, H))) for _ in range(L)]
        h_der = [pin(torch.empty((n, H))) for _ in range(L)]
        arena = torch.empty(B.sar_gat_stack_arena_bytes(g.whole, L, H, F, B._dtype(feat0)), dtype=torch.uint8, device=DEV)
        B.sar_gat_stack_host(g.whole, g.bounds, H, F, cfg.slope, pin(feat0), [pin(x) for x in els],
                             [pin(x) for x in ers], pin(gout), h_out, h_dfeat, h_del, h_der, arena)
        torch.cuda.synchronize()
        # the same chain with device tensors
        x = feat0.to(DEV)
        saved = []
        for l in range(L):
            o, m, d = api.gat_forward(g, x, els[l].to(DEV), ers[l].to(DEV), cfg.slope)
            saved.append((x, m, d))
            x = o
        assert torch.equal(x.cpu(), h_out)
        gr = gout.to(DEV)
        for l in reversed(range(L)):
            xin, m, d = saved[l]
            gr, dl, dr = api.gat_backward(g, xin, els[l].to(DEV), ers[l].to(DEV), m, d, gr, cfg.slope)
            assert torch.equal(dl.cpu(), h_del[l]) and torch.equal(dr.cpu(), h_der[l])
        assert torch.equal(gr.cpu(), h_dfeat)


def test_stack_host_pipelined_calls_equal_plain_calls():
    """Five pipelined calls with different inputs (two working sets used alternately, copies of one call
    overlapping the kernels of the previous one) return what five plain calls return, then a plain call
    after them still works."""
    from paper_2111_06483_b200 import binding as B
    cfg = workloads.CONFIGS["seqpart"].scaled(0.5)
    n, H, F, L, T = cfg.n, cfg.heads, cfg.feat, 2, 5
    src, dst = workloads.make_graph(cfg, device=DEV)
    g = api.Graph.from_coo(n, src, dst, k=cfg.k)
    tdt = torch.bfloat16
    pin = lambda x: x.pin_memory()
    ins = []
    for t in range(T):
        ins.append(dict(
            feat0=pin(workloads.normal_tensor((n, H, F), 50 + t, 10, dtype=tdt)),
            gout=pin(workloads.normal_tensor((n, H, F), 50 + t, 11, dtype=tdt)),
            el=[pin(workloads.normal_tensor((n, H), 50 + t, 16 * l + 12)) for l in range(L)],
            er=[pin(workloads.normal_tensor((n, H), 50 + t, 16 * l + 13)) for l in range(L)]))

    def outputs():
        return dict(out=pin(torch.empty((n, H, F), dtype=tdt)), dfeat=pin(torch.empty((n, H, F), dtype=tdt)),
                    del_=[pin(torch.empty((n, H))) for _ in range(L)], der=[pin(torch.empty((n, H))) for _ in range(L)])

    one = B.sar_gat_stack_arena_bytes(g.whole, L, H, F, B.SAR_BF16)
    arena = torch.empty(2 * ((one + 255) // 256 * 256), dtype=torch.uint8, device=DEV)

    def call(i, o, pipelined):
        B.sar_gat_stack_host(g.whole, g.bounds, H, F, cfg.slope, i["feat0"], i["el"], i["er"], i["gout"], o["out"],
                             o["dfeat"], o["del_"], o["der"], arena, pipelined=pipelined)

    plain = [outputs() for _ in range(T)]
    for t in range(T):
        call(ins[t], plain[t], False)
    torch.cuda.synchronize()
    piped = [outputs() for _ in range(T)]
    for t in range(T):
        call(ins[t], piped[t], True)
    B.sar_gat_stack_host_wait()
    torch.cuda.synchronize()
    for t in range(T):
        assert torch.equal(piped[t]["out"], plain[t]["out"]) and torch.equal(piped[t]["dfeat"], plain[t]["dfeat"]), t
        for l in range(L):
            assert torch.equal(piped[t]["del_"][l], plain[t]["del_"][l]), (t, l)
            assert torch.equal(piped[t]["der"][l], plain[t]["der"][l]), (t, l)
    assert not torch.equal(plain[0]["out"], plain[1]["out"])
    again = outputs()
    call(ins[2], again, False)  # switching back to the plain mode
    torch.cuda.synchronize()
    assert torch.equal(again["out"], plain[2]["out"]) and torch.equal(again["dfeat"], plain[2]["dfeat"])
    with pytest.raises(B.SarError) as ei:  # the pipelined mode needs both working sets
        B.sar_gat_stack_host(g.whole, g.bounds, H, F, cfg.slope, ins[0]["feat0"], ins[0]["el"], ins[0]["er"],
                             ins[0]["gout"], again["out"], again["dfeat"], again["del_"], again["der"],
                             arena[:one], pipelined=True)
    assert ei.value.code == -4


def test_more_than_two_to_the_31_edges():
    """Maximum sizes: an edge count that does not fit 32 bits (edge offsets are 64-bit throughout).  No oracle
    can visit 2.3 G edges in test time, so the checks are the ones that hold at any size: the CSR's degrees
    equal a count of the destination ids made with torch, the library's own scan finds it well formed, the
    sum of an all-ones feature is the degree (exact in float32 below 2^24), and an attention layer over
    constant features returns that constant with d = degree and m = 0 when all scores are zero."""
    from paper_2111_06483_b200 import binding as B
    if torch.cuda.get_device_properties(0).total_memory < 120e9:
        pytest.skip("needs about 90 GB of device memory")
    n, e = 2_000_000, (1 << 31) + (1 << 27)
    spec = workloads.ChungLuSpec(n=n, e=e, gamma=2.1, d_max=100_000.0, seed=31)
    src, dst = workloads.chung_lu_edges(spec, device=DEV)
    deg = torch.zeros(n, dtype=torch.int64, device=DEV)
    for lo in range(0, e, 1 << 28):
        deg += torch.bincount(dst[lo:lo + (1 << 28)].long(), minlength=n)
    g = api.Graph.from_coo(n, src, dst, k=1)
    del src, dst
    torch.cuda.empty_cache()
    assert g.nnz == e and int(g.whole.indptr[-1]) == e and e > 2 ** 31
    assert torch.equal(g.whole.indptr[1:] - g.whole.indptr[:-1], deg)
    assert int((g.whole.t_indptr[1:] - g.whole.t_indptr[:-1]).sum()) == e
    flag = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.sar_validate_part(g.whole, flag)  # raises on a malformed CSR / CSC
    assert int(deg.max()) < 2 ** 24
    ones = torch.ones((n, 8), dtype=torch.float32, device=DEV)
    assert torch.equal(api.spmm_sum(g.whole, ones), deg.float()[:, None].expand(n, 8))
    # the rows at the far end of the edge array in particular
    tail = torch.nonzero(g.whole.indptr[:-1] > 2 ** 31).flatten()
    assert tail.numel() > 1000
    H, F = 2, 8
    feat = torch.full((n, H, F), 3.0, dtype=torch.float32, device=DEV)
    zeros = torch.zeros((n, H), dtype=torch.float32, device=DEV)
    out, m, d = api.gat_forward(g, feat, zeros, zeros, 0.2)
    has = deg > 0
    assert torch.equal(d, deg.float()[:, None].expand(n, H))
    assert torch.equal(m[has], torch.zeros_like(m[has])) and bool(torch.isinf(m[~has]).all())
    want = torch.where(has[:, None, None], torch.full_like(out, 3.0), torch.zeros_like(out))
    assert float((out - want).abs().max()) <= 3.0 * 1e-5
    # backward: with constant features every d(alpha) equals D, so del = der = 0, and sum_j dfeat[j] = sum_i gout[i] over the rows with edges
    gout = torch.ones_like(feat)
    dfeat, del_, der = api.gat_backward(g, feat, zeros, zeros, m, d, gout, 0.2)
    assert float(del_.abs().max()) <= 1e-3 and float(der.abs().max()) <= 1e-3
    total = float(dfeat[:, 0, 0].double().sum())
    assert abs(total - float(has.sum())) <= 1e-4 * float(has.sum())   # sum_j dfeat[j] = number of rows with edges
    del g, feat, out, dfeat
    torch.cuda.empty_cache()
